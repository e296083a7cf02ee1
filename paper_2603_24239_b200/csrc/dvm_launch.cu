// Launch side of libdvm: sends a bytecode program to the device (as the kernel-parameter block)
// and starts the virtual machine on a persistent grid.
#include <cuda_runtime.h>
#include <stdio.h>
#include <string.h>

#include <mutex>
#include <unordered_map>

#include "../../include/dvm.h"
#include "dvm_format.h"
#include "dvm_internal.h"
#include "dvm_launch.h"
#include "dvm_vm.cuh"
#include "dvm_vm_variants.h"

namespace {

constexpr int PW_SMALL = DVM_PW_SMALL;
constexpr int PW_LARGE = DVM_PW_LARGE;
constexpr int QUEUE_SLOTS = 504;
constexpr size_t SCRATCH_BYTES = (8 + 4 * QUEUE_SLOTS) * sizeof(unsigned int);
constexpr int MAX_DEVICES = 64;
constexpr size_t kMaxDynSmem = 227 * 1024 - 9 * 1024;  // dynamic shared memory a CTA may ask for (8.3 KB static part excluded)

struct DeviceState {
  bool ready = false;
  unsigned int* scratch = nullptr;  // [0] status word, [8 + 4*slot] work-queue counters (next tile, CTAs finished, tiles completed)
  int sm_count = 0;
  // resident CTAs per SM, per (kernel variant, bytes of dynamic shared memory / DVM_LOCAL_UNIT): occupancy depends
  // on exactly these two, so a one-slot and a two-slot launch of the same program never share an entry
  std::unordered_map<uint64_t, int> occ;
  unsigned queue_slot = 0;
};

DeviceState g_dev[MAX_DEVICES];
std::mutex g_mu;
thread_local int t_last_cuda_error = 0;
long long g_launches = 0;

}  // namespace

int dvm_device_state(DvmDeviceInfo* info) {
  int dev = 0;
  DVM_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return DVM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_mu);
  DeviceState& d = g_dev[dev];
  if (!d.ready) {
    DVM_CUDA(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
    DVM_CUDA(cudaMalloc(&d.scratch, SCRATCH_BYTES));
    DVM_CUDA(cudaMemset(d.scratch, 0, SCRATCH_BYTES));
    d.ready = true;
  }
  info->scratch = d.scratch;
  info->sm_count = d.sm_count;
  info->queue_slot = d.queue_slot;
  d.queue_slot = (d.queue_slot + 1) % QUEUE_SLOTS;
  return DVM_OK;
}

// The groups of interpreter variants (dvm_vm_inst.cu, compiled once per group).
#define DVM_GROUPS(X) X(0) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12)
#define DVM_DECL_GROUP(g) const DvmVmVariant* dvm_vm_group_##g(int* count);
DVM_GROUPS(DVM_DECL_GROUP)
#undef DVM_DECL_GROUP

const DvmVmVariant* dvm_vm_find_variant(int V, bool large, bool single, int ext, bool levels) {
  typedef const DvmVmVariant* (*GroupFn)(int*);
#define DVM_GROUP_FN(g) &dvm_vm_group_##g,
  static const GroupFn groups[] = {DVM_GROUPS(DVM_GROUP_FN)};
#undef DVM_GROUP_FN
  for (GroupFn g : groups) {
    int n = 0;
    const DvmVmVariant* v = g(&n);
    for (int i = 0; i < n; ++i)
      if (v[i].V == V && v[i].large == (int)large && v[i].single == (int)single && v[i].ext == ext && v[i].levels == (int)levels)
        return &v[i];
  }
  return nullptr;
}

// Key of the occupancy cache: the variant and the dynamic shared memory in local-memory units.
uint64_t dvm_occupancy_key(const DvmVmVariant* v, size_t smem) {
  const uint64_t id = (uint64_t)v->V | ((uint64_t)v->large << 8) | ((uint64_t)v->single << 9) | ((uint64_t)v->ext << 10) |
                      ((uint64_t)v->levels << 12);
  return (id << 32) | (uint64_t)(smem / DVM_LOCAL_UNIT);
}

// Resident CTAs per SM of one interpreter variant for a launch with `smem` bytes of dynamic shared memory
// (cached per device).  The variants with level waits rely on the whole grid being resident: no CTA fits -> no launch.
static int dvm_occupancy(const DvmVmVariant* v, size_t smem, int* out) {
  int dev = 0;
  DVM_CUDA(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lk(g_mu);
  DeviceState& d = g_dev[dev];
  const uint64_t key = dvm_occupancy_key(v, smem);
  auto it = d.occ.find(key);
  if (it == d.occ.end()) {
    int n = 0;
    DVM_CUDA(v->occupancy(smem, kMaxDynSmem, &n));
    if (n <= 0) {
      if (v->levels) return DVM_ERR_TOO_LARGE;
      n = 1;
    }
    it = d.occ.emplace(key, n).first;
  }
  *out = it->second;
  return DVM_OK;
}

void dvm_note_cuda_error(int e) { t_last_cuda_error = e; }
void dvm_count_launch() { __atomic_add_fetch(&g_launches, 1, __ATOMIC_RELAXED); }

extern "C" int dvm_last_cuda_error(void) { return t_last_cuda_error; }
extern "C" int64_t dvm_launch_count(void) { return (int64_t)__atomic_load_n(&g_launches, __ATOMIC_RELAXED); }

namespace {

// Copies one verified vector program into `dst` and patches in what only the launch knows: the tensor
// addresses, each input register's address phase (address modulo 16), and -- when the program assumed
// 16-byte aligned rows but the primary operand's base pointer is not -- the switch to address-derived shifts.
int place_program(uint32_t* dst, const uint32_t* code, void* const* tensors, int n_tensors) {
  const uint32_t total = code[DVM_H_TOTAL_WORDS];
  memcpy(dst, code, (size_t)total * 4);
  const uint32_t counts = code[DVM_H_COUNTS];
  const uint32_t nt = counts & 0xff, n_opd = (counts >> 16) & 0xff;
  if ((uint32_t)n_tensors != nt) return DVM_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < nt; ++i) {
    if (!tensors[i]) return DVM_ERR_INVALID_ARG;
    unsigned long long a = (unsigned long long)(uintptr_t)tensors[i];
    dst[DVM_HDR_WORDS + 2 * i] = (uint32_t)a;
    dst[DVM_HDR_WORDS + 2 * i + 1] = (uint32_t)(a >> 32);
  }
  const uint32_t* ot = code + DVM_HDR_WORDS + 2 * nt;
  for (uint32_t o = 0; o < n_opd; ++o) {
    uint32_t info = ot[o * DVM_OPD_WORDS];
    uintptr_t a = (uintptr_t)tensors[info & 0xff];
    uintptr_t es = ((info >> 8) & 0xff) == DVM_DT_BF16 ? 2 : 4;
    if (a % es) return DVM_ERR_INVALID_ARG;
  }
  // every input register learns its tensor's address modulo 16 (the images keep that phase)
  {
    const uint32_t n_inr = code[DVM_H_LOCAL] & 0xff;
    uint32_t* lt = dst + DVM_HDR_WORDS + 2 * nt + n_opd * DVM_OPD_WORDS;
    for (uint32_t k = 0; k < n_inr; ++k) {
      const uint32_t info = ot[(lt[k] >> 24) * DVM_OPD_WORDS];
      lt[k] = (lt[k] & ~(0xfu << 20)) | (((uint32_t)(uintptr_t)tensors[info & 0xff] & 15u) << 20);
    }
  }
  // A program encoded for aligned rows relies on a 16-byte aligned primary tensor; on any other base address
  // the interpreter derives the row shift from the actual address instead (the rows' last columns then
  // wrap around into the head slots when a row fills its whole capacity).
  const uint32_t geom = code[DVM_H_GEOM];
  const uint32_t flags = geom >> 24;
  if ((flags & DVM_F_ALIGNED) && code[DVM_H_PRIMARY] != 0xffffffffu) {
    const uint32_t info = ot[code[DVM_H_PRIMARY] * DVM_OPD_WORDS];
    if (((uintptr_t)tensors[info & 0xff]) & 15) dst[DVM_H_GEOM] = geom & ~((uint32_t)DVM_F_ALIGNED << 24);
  }
  return DVM_OK;
}

// Results that tiles combine atomically start from the operation's identity.
__global__ void dvm_fill_kernel(uint32_t* p, uint32_t n, uint32_t bits) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) p[i] = bits;
}

int prefill_combined(const uint32_t* code, void* const* tensors, cudaStream_t stream) {
  const uint32_t counts = code[DVM_H_COUNTS];
  const uint32_t nt = counts & 0xff, n_opd = (counts >> 16) & 0xff;
  const uint32_t* ot = code + DVM_HDR_WORDS + 2 * nt;
  for (uint32_t o = 0; o < n_opd; ++o) {
    const uint32_t info = ot[o * DVM_OPD_WORDS + DVM_OPD_INFO], comb = (info >> 26) & 3u;
    if (!comb) continue;
    const uint32_t n = ot[o * DVM_OPD_WORDS + DVM_OPD_FILL];
    if (n == 0) continue;
    const uint32_t bits = comb == 1 ? 0u : (comb == 2 ? 0xff800000u : 0x7f800000u);  // 0, -inf, +inf
    const int blocks = (int)((n + 255u) / 256u < 1184u ? (n + 255u) / 256u : 1184u);
    dvm_fill_kernel<<<blocks, 256, 0, stream>>>(static_cast<uint32_t*>(tensors[info & 0xff]), n, bits);
    DVM_CUDA(cudaGetLastError());
    dvm_count_launch();
  }
  return DVM_OK;
}

int prefill_all(int n_programs, const void* const* codes, void* const* const* tensors, cudaStream_t stream) {
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t* c = (const uint32_t*)codes[i];
    if (!((c[DVM_H_GEOM] >> 24) & DVM_F_VIEWS)) continue;
    int st = prefill_combined(c, tensors[i], stream);
    if (st != DVM_OK) return st;
  }
  return DVM_OK;
}

// Starts one interpreter variant on `grid` CTAs.
int launch_variant(const DvmVmVariant* v, const void* params, int grid, size_t smem, cudaStream_t stream) {
  DVM_CUDA(v->launch(params, grid, smem, stream));
  dvm_count_launch();
  return DVM_OK;
}

// The variant a launch needs: 24 elements per thread exist as the one-program basic variant only.
const DvmVmVariant* pick_variant(int V, bool large, bool single, int ext, bool levels) {
  if (levels) single = false;
  return dvm_vm_find_variant(V, large, single, ext, levels);
}

thread_local dvm::VMParams<PW_LARGE> t_large;  // 32 KB, reused by every launch of the thread

// `level` (may be NULL): level[i] of program i, non-decreasing; a program reads what programs of lower levels store.
int launch_vec(int n_programs, const void* const* codes, void* const* const* tensors, const int* n_tensors,
               bool use_queue, const int* level, cudaStream_t stream) {
  // A program that asks for a single tile slot (DVM_F_ONE_SLOT), launched on its own: the variant with level
  // waits runs it, every tile held back until the CTA's previous tile is done, nothing waited for.
  const bool one_slot = n_programs == 1 && !level &&
                        ((((const uint32_t*)codes[0])[DVM_H_GEOM] >> 24) & DVM_F_ONE_SLOT) != 0;
  static const int kOneLevel[1] = {0};
  if (one_slot) { level = kOneLevel; use_queue = true; }
  // directory: [program word offsets (n)][tile prefix sums (n+1)][tiles before the program's level (n, with levels)]
  uint32_t dir = (level ? 3 : 2) * (uint32_t)n_programs + 1;
  uint64_t need = dir;
  uint64_t total_tiles = 0;
  uint32_t units = 0;
  int V = 0;
  int ext = 0;  // the extension level the launch needs: 1 Cmp / Select / Pow / IsFinite, 2 also views
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t* c = (const uint32_t*)codes[i];
    need += c[DVM_H_TOTAL_WORDS];
    total_tiles += c[DVM_H_N_TILES];
    if ((c[DVM_H_LOCAL2] >> 16) > units) units = c[DVM_H_LOCAL2] >> 16;
    const int v = (int)(c[DVM_H_LOCAL] >> 24);
    if (((c[DVM_H_GEOM] >> 24) & DVM_F_EXT_ISA) && ext < 1) ext = 1;
    if ((c[DVM_H_GEOM] >> 24) & DVM_F_VIEWS) ext = 2;
    if (V && v != V) return DVM_ERR_INVALID_ARG;  // one kernel variant per launch: same elements per thread
    V = v;
  }
  if (need > PW_LARGE || total_tiles > 0xffffffffull) return DVM_ERR_TOO_LARGE;
  if (total_tiles == 0) return DVM_OK;

  DvmDeviceInfo dev;
  int st = dvm_device_state(&dev);
  if (st != DVM_OK) return st;

  dvm::VMParams<PW_LARGE>& P = t_large;
  uint32_t pos = dir, tb = 0, level_start = 0;
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t* c = (const uint32_t*)codes[i];
    P.words[i] = pos;
    P.words[n_programs + i] = tb;
    if (level) {
      if (i > 0 && level[i] != level[i - 1]) level_start = tb;  // every tile before this one belongs to a lower level
      P.words[2 * n_programs + 1 + i] = level_start;
    }
    st = place_program(P.words + pos, c, tensors[i], n_tensors[i]);
    if (st != DVM_OK) return st;
    pos += c[DVM_H_TOTAL_WORDS];
    tb += c[DVM_H_N_TILES];
  }
  P.words[2 * n_programs] = tb;
  P.n_programs = (uint32_t)n_programs;
  P.total_tiles = (uint32_t)total_tiles;
  P.n_words = pos;
  P.use_queue = use_queue ? 1u : 0u;
  P.levels = one_slot ? 2u : (level ? 1u : 0u);
  P.status = dev.scratch;
  P.queue = dev.scratch + 8 + 4 * dev.queue_slot;

  const bool large = pos > PW_SMALL;
  const size_t smem = ((one_slot ? 1 : 2) * (size_t)units + 1) * DVM_LOCAL_UNIT;  // one spare unit, two tile slots (or one)
  P.slot_bytes = one_slot ? 0u : units * DVM_LOCAL_UNIT;
  if (smem > kMaxDynSmem) return DVM_ERR_TOO_LARGE;
  const bool single = n_programs == 1 && !use_queue;
  const DvmVmVariant* variant = pick_variant(V, large, single, ext, level != nullptr);
  if (!variant) return DVM_ERR_UNSUPPORTED;  // (24 elements per thread: encoded for a launch of its own on the basic variant)
  int occ = 0;
  st = dvm_occupancy(variant, smem, &occ);
  if (st != DVM_OK) return st;
  uint64_t slots = (uint64_t)dev.sm_count * occ;
  int grid = (int)(total_tiles < slots ? total_tiles : slots);
  // Everything is placed and checked: only now touch the caller's memory.  Results that tiles combine
  // atomically are filled with their identity (one small kernel per such output), then the interpreter starts.
  st = prefill_all(n_programs, codes, tensors, stream);
  if (st != DVM_OK) return st;
  if (!large) {
    dvm::VMParams<PW_SMALL> S;
    memcpy(&S, &P, offsetof(dvm::VMParams<PW_SMALL>, words) + (size_t)pos * 4);
    return launch_variant(variant, &S, grid, smem, stream);
  }
  return launch_variant(variant, &P, grid, smem, stream);
}

}  // namespace

extern "C" int dvm_launch(const void* code, size_t code_size, void* const* tensors, int n_tensors,
                          void* cuda_stream) {
  if (!code || !tensors) return DVM_ERR_INVALID_ARG;
  int st = dvm_verify(code, code_size);
  if (st != DVM_OK) return st;
  const uint32_t* w = (const uint32_t*)code;
  if (w[DVM_H_KERNEL_TYPE] == DVM_KERNEL_MATMUL)
    return dvm_launch_matmul(w, code_size / 4, tensors, n_tensors, (cudaStream_t)cuda_stream);
  const void* codes[1] = {code};
  void* const* tl[1] = {tensors};
  return launch_vec(1, codes, tl, &n_tensors, false, nullptr, (cudaStream_t)cuda_stream);
}

extern "C" int dvm_launch_stacked(int n_programs, const void* const* codes, const size_t* code_sizes,
                                  void* const* const* tensors, const int* n_tensors, void* cuda_stream) {
  if (n_programs < 0 || (n_programs > 0 && (!codes || !code_sizes || !tensors || !n_tensors)))
    return DVM_ERR_INVALID_ARG;
  if (n_programs == 0) return DVM_OK;
  if (n_programs > DVM_MAX_STACK) return DVM_ERR_TOO_LARGE;
  for (int i = 0; i < n_programs; ++i) {
    if (!codes[i] || !tensors[i]) return DVM_ERR_INVALID_ARG;
    int st = dvm_verify(codes[i], code_sizes[i]);
    if (st != DVM_OK) return st;
    // only vector meta-kernels stack (Sec. 5.1: stacking of meta-kernels on the Vector units)
    if (((const uint32_t*)codes[i])[DVM_H_KERNEL_TYPE] != DVM_KERNEL_VEC) return DVM_ERR_UNSUPPORTED;
  }
  return launch_vec(n_programs, codes, tensors, n_tensors, true, nullptr, (cudaStream_t)cuda_stream);
}

extern "C" int dvm_launch_stacked_levels(int n_programs, const void* const* codes, const size_t* code_sizes,
                                         void* const* const* tensors, const int* n_tensors, const int* level,
                                         void* cuda_stream) {
  if (n_programs < 0 || (n_programs > 0 && (!codes || !code_sizes || !tensors || !n_tensors || !level)))
    return DVM_ERR_INVALID_ARG;
  if (n_programs == 0) return DVM_OK;
  if (n_programs > DVM_MAX_STACK) return DVM_ERR_TOO_LARGE;
  for (int i = 0; i < n_programs; ++i) {
    if (!codes[i] || !tensors[i]) return DVM_ERR_INVALID_ARG;
    if (i > 0 && level[i] < level[i - 1]) return DVM_ERR_INVALID_ARG;  // the work queue hands tiles out in level order
    int st = dvm_verify(codes[i], code_sizes[i]);
    if (st != DVM_OK) return st;
    if (((const uint32_t*)codes[i])[DVM_H_KERNEL_TYPE] != DVM_KERNEL_VEC) return DVM_ERR_UNSUPPORTED;
  }
  return launch_vec(n_programs, codes, tensors, n_tensors, true, level, (cudaStream_t)cuda_stream);
}

extern "C" int dvm_run_host(const void* code, size_t code_size, void* const* host_tensors,
                            const size_t* tensor_bytes, int n_tensors, void* staging, size_t staging_bytes,
                            void* cuda_stream) {
  if (!code || !host_tensors || !tensor_bytes || !staging) return DVM_ERR_INVALID_ARG;
  int st = dvm_verify(code, code_size);
  if (st != DVM_OK) return st;
  const uint32_t* w = (const uint32_t*)code;
  const uint32_t counts = w[DVM_H_COUNTS];
  const int nt = counts & 0xff, n_in = (counts >> 8) & 0xff;
  if (n_tensors != nt || nt > DVM_MAX_TENSORS) return DVM_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  void* dev[DVM_MAX_TENSORS];
  size_t off = 0;
  for (int i = 0; i < nt; ++i) {
    dev[i] = (char*)staging + off;
    off += (tensor_bytes[i] + 255) & ~(size_t)255;
  }
  if (off > staging_bytes) return DVM_ERR_BUFFER_TOO_SMALL;
  for (int i = 0; i < n_in; ++i)
    if (tensor_bytes[i]) DVM_CUDA(cudaMemcpyAsync(dev[i], host_tensors[i], tensor_bytes[i], cudaMemcpyHostToDevice, stream));
  st = dvm_launch(code, code_size, dev, nt, cuda_stream);
  if (st != DVM_OK) return st;
  for (int i = n_in; i < nt; ++i)
    if (tensor_bytes[i]) DVM_CUDA(cudaMemcpyAsync(host_tensors[i], dev[i], tensor_bytes[i], cudaMemcpyDeviceToHost, stream));
  DVM_CUDA(cudaStreamSynchronize(stream));
  return DVM_OK;
}

// ---- self-test of the bounded waits ----
namespace {
__global__ void dvm_selftest_vm_wait_kernel(unsigned int* status) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = static_cast<uint32_t>(__cvta_generic_to_shared(&bar));
  if (threadIdx.x == 0) {
    dvm::vm_mbar_init(b, 2);  // two arrivals expected, one ever made: the phase never completes
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    dvm::vm_mbar_arrive(b);
  }
  __syncthreads();
  if (!dvm::vm_mbar_wait(b, 0) && threadIdx.x == 0) atomicMax(status, (unsigned int)dvm::ST_TIMEOUT);
}
// The level wait of dvm_launch_stacked_levels on a counter nobody advances (the status word's neighbour,
// which stays zero): it gives up after its limit.
__global__ void dvm_selftest_level_wait_kernel(unsigned int* status) {
  if (threadIdx.x == 0 && !dvm::vm_wait_tiles_done(status + 1, 1u)) atomicMax(status, (unsigned int)dvm::ST_TIMEOUT);
}
}  // namespace

int dvm_selftest_mm_wait(unsigned int* status, cudaStream_t stream);

extern "C" int dvm_selftest_bounded_wait(int which, void* cuda_stream) {
  DvmDeviceInfo dev;
  int st = dvm_device_state(&dev);
  if (st != DVM_OK) return st;
  if (which == 0) {
    dvm_selftest_vm_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(dev.scratch);
    DVM_CUDA(cudaGetLastError());
    dvm_count_launch();
    return DVM_OK;
  }
  if (which == 1) return dvm_selftest_mm_wait(dev.scratch, (cudaStream_t)cuda_stream);
  if (which == 2) {
    dvm_selftest_level_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(dev.scratch);
    DVM_CUDA(cudaGetLastError());
    dvm_count_launch();
    return DVM_OK;
  }
  return DVM_ERR_INVALID_ARG;
}

extern "C" int dvm_last_device_status(void* cuda_stream, int* status) {
  if (!status) return DVM_ERR_INVALID_ARG;
  DVM_CUDA(cudaStreamSynchronize((cudaStream_t)cuda_stream));
  DvmDeviceInfo dev;
  int st = dvm_device_state(&dev);
  if (st != DVM_OK) return st;
  unsigned int v = 0;
  DVM_CUDA(cudaMemcpy(&v, dev.scratch, 4, cudaMemcpyDeviceToHost));
  if (v) DVM_CUDA(cudaMemset(dev.scratch, 0, 4));
  *status = v == dvm::ST_OK ? DVM_OK : (v == dvm::ST_TIMEOUT ? DVM_ERR_DEVICE_TIMEOUT : DVM_ERR_DEVICE_BAD_CODE);
  return DVM_OK;
}

// ---------------------------------------------------------------------------------------------
// dvm_launch_stacked_noalloc: the stacked launch for callers that must not allocate device memory.
//
// dvm_launch_stacked keeps its work-queue counters in a small buffer that the library obtains with
// cudaMalloc the first time a device is used.  Some callers cannot tolerate that: code running inside a
// memory pool or arena that owns every byte of the device, latency-critical serving loops where a first-use
// cudaMalloc (an implicit device synchronisation) is unacceptable, and sandboxes that forbid the allocator
// outright.  For them the same kernel runs with its queue in the fixed array below, which is part of the
// library image: every GPU that loads the library holds these 256 bytes until the process exits.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int NOALLOC_WORDS = 64;                 // 256 bytes: [0] status word, [2..4] work-queue counters
static __device__ __align__(256) unsigned int dvm_noalloc_scratch[NOALLOC_WORDS];

struct NoAllocDevice {
  unsigned int* scratch = nullptr;  // device address of dvm_noalloc_scratch on this device
  int sm_count = 0;
};
NoAllocDevice g_noalloc[MAX_DEVICES];
std::mutex g_noalloc_mu;

// Once per device, with that device current: resolve the array's device address.  In host code the array's
// name is only a stand-in for the symbol; the address a kernel may use comes from cudaGetSymbolAddress.
int noalloc_device(NoAllocDevice* out) {
  int dev = 0;
  DVM_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return DVM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_noalloc_mu);
  NoAllocDevice& d = g_noalloc[dev];
  if (!d.scratch) {
    void* p = nullptr;
    DVM_CUDA(cudaGetSymbolAddress(&p, dvm_noalloc_scratch));
    DVM_CUDA(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
    d.scratch = static_cast<unsigned int*>(p);
  }
  *out = d;
  return DVM_OK;
}

}  // namespace

extern "C" int dvm_launch_stacked_noalloc(int n_programs, const void* const* codes, const size_t* code_sizes,
                                          void* const* const* tensors, const int* n_tensors, void* cuda_stream) {
  if (n_programs < 0 || (n_programs > 0 && (!codes || !code_sizes || !tensors || !n_tensors)))
    return DVM_ERR_INVALID_ARG;
  if (n_programs == 0) return DVM_OK;
  if (n_programs > DVM_NOALLOC_MAX_PROGRAMS) return DVM_ERR_TOO_LARGE;  // beyond the stated maximum
  uint32_t dir = 2 * (uint32_t)n_programs + 1;
  uint64_t need = dir, total_tiles = 0;
  uint32_t units = 0;
  int V = 0;
  int ext = 0;  // the extension level the launch needs: 1 Cmp / Select / Pow / IsFinite, 2 also views
  for (int i = 0; i < n_programs; ++i) {
    if (!codes[i] || !tensors[i]) return DVM_ERR_INVALID_ARG;
    int st = dvm_verify(codes[i], code_sizes[i]);
    if (st != DVM_OK) return st;
    const uint32_t* c = (const uint32_t*)codes[i];
    if (c[DVM_H_KERNEL_TYPE] != DVM_KERNEL_VEC) return DVM_ERR_UNSUPPORTED;
    need += c[DVM_H_TOTAL_WORDS];
    total_tiles += c[DVM_H_N_TILES];
    if ((c[DVM_H_LOCAL2] >> 16) > units) units = c[DVM_H_LOCAL2] >> 16;
    const int v = (int)(c[DVM_H_LOCAL] >> 24);
    if (((c[DVM_H_GEOM] >> 24) & DVM_F_EXT_ISA) && ext < 1) ext = 1;
    if ((c[DVM_H_GEOM] >> 24) & DVM_F_VIEWS) ext = 2;
    if (V && v != V) return DVM_ERR_INVALID_ARG;
    V = v;
  }
  if (need > PW_LARGE || total_tiles > DVM_NOALLOC_MAX_TILES) return DVM_ERR_TOO_LARGE;
  if (total_tiles == 0) return DVM_OK;

  NoAllocDevice dev;
  int st = noalloc_device(&dev);
  if (st != DVM_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  dvm::VMParams<PW_LARGE>& P = t_large;
  uint32_t pos = dir, tb = 0;
  for (int i = 0; i < n_programs; ++i) {
    const uint32_t* c = (const uint32_t*)codes[i];
    P.words[i] = pos;
    P.words[n_programs + i] = tb;
    st = place_program(P.words + pos, c, tensors[i], n_tensors[i]);
    if (st != DVM_OK) return st;
    pos += c[DVM_H_TOTAL_WORDS];
    tb += c[DVM_H_N_TILES];
  }
  P.words[2 * n_programs] = tb;
  P.n_programs = (uint32_t)n_programs;
  P.total_tiles = (uint32_t)total_tiles;
  P.n_words = pos;
  P.use_queue = 1u;
  P.levels = 0u;
  P.status = dev.scratch;
  P.queue = dev.scratch + 2;
  const size_t smem = (2 * (size_t)units + 1) * DVM_LOCAL_UNIT;
  P.slot_bytes = units * DVM_LOCAL_UNIT;
  if (smem > kMaxDynSmem) return DVM_ERR_TOO_LARGE;
  const bool large = pos > PW_SMALL;
  const DvmVmVariant* variant = pick_variant(V, large, false, ext, false);
  if (!variant) return DVM_ERR_UNSUPPORTED;
  int occ = 0;
  st = dvm_occupancy(variant, smem, &occ);
  if (st != DVM_OK) return st;
  uint64_t slots = (uint64_t)dev.sm_count * occ;
  int grid = (int)(total_tiles < slots ? total_tiles : slots);
  // every call shares the array and it keeps the last call's contents: the queue counters must start at zero
  DVM_CUDA(cudaMemsetAsync(dev.scratch, 0, NOALLOC_WORDS * sizeof(unsigned int), stream));
  st = prefill_all(n_programs, codes, tensors, stream);
  if (st != DVM_OK) return st;
  if (!large) {
    dvm::VMParams<PW_SMALL> S;
    memcpy(&S, &P, offsetof(dvm::VMParams<PW_SMALL>, words) + (size_t)pos * 4);
    return launch_variant(variant, &S, grid, smem, stream);
  }
  return launch_variant(variant, &P, grid, smem, stream);
}
