/* libdvm -- C ABI of the B200-native bytecode virtual machine for fused dynamic
 * tensor operators.
 *
 * The calls follow the paper's statement of the problem (Sec. 3 "Operator
 * Compiler", Sec. 4): given a computation graph of basic operators to fuse and
 * the concrete input shapes of one instance, the host encodes a bytecode
 * program (dvm_encode); the program is sent to the device, where a virtual
 * machine decodes it into tile-level virtual instructions and executes them
 * over the tiles of the runtime shape (dvm_launch); several independent
 * meta-kernels may be stacked into one kernel (dvm_launch_stacked, Sec. 5.1
 * "Stacking-based fusion").  Nothing is cached between instances.
 *
 * Conventions
 *  - Every call returns an int status: DVM_OK (0) or a negative DVM_ERR_*.
 *    No exception crosses the boundary, nothing traps.
 *  - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global
 *    memory of the current device.  The library never allocates, frees or
 *    copies tensor memory and never synchronises a stream (dvm_run_host and
 *    dvm_last_device_status are the documented exceptions).
 *  - Tensors are dense row-major.  A dimension of size 1 broadcasts
 *    numpy-style (right-aligned) against the other operands.
 *  - Bytecode refers to tensor *slots* (inputs in declaration order, then
 *    outputs in declaration order); device addresses are supplied at launch, so
 *    one encoded program can be launched on any buffers of the encoded shapes.
 */
#ifndef DVM_H_
#define DVM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DVM_MAX_RANK 6

enum {
  DVM_OK = 0,
  DVM_ERR_INVALID_ARG = -1,      /* NULL pointer, bad id / enum, bad rank, misaligned element pointer */
  DVM_ERR_SHAPE_MISMATCH = -2,   /* operands do not broadcast, matmul inner dims differ */
  DVM_ERR_UNSUPPORTED = -3,      /* valid program the VM cannot run (row longer than the register
                                    budget, too many live values, more than 3 non-mergeable outer dims) */
  DVM_ERR_BUFFER_TOO_SMALL = -4, /* code buffer too small; *code_size receives the need */
  DVM_ERR_BAD_CODE = -5,         /* bytecode failed verification */
  DVM_ERR_CUDA = -6,             /* a CUDA runtime call failed; see dvm_last_cuda_error */
  DVM_ERR_DEVICE_TIMEOUT = -7,   /* a bounded device-side wait ran out (status word) */
  DVM_ERR_DEVICE_BAD_CODE = -8,  /* the interpreter met an instruction it cannot decode (status word) */
  DVM_ERR_NOT_FINALIZED = -9,
  DVM_ERR_TOO_LARGE = -10        /* program / stack exceeds a fixed library limit */
};

/* Element types.  U8 and I32 are for outputs and for dvm_program_cast (Table 1, Cast; a Cmp / IsFinite result is
 * stored as 0 / 1): the fp32 value is converted toward zero, values outside the type's range take the nearest
 * bound, NaN gives 0.  Inputs are F32 or BF16. */
enum { DVM_F32 = 0, DVM_BF16 = 1, DVM_U8 = 2, DVM_I32 = 3 };

/* Unary operators.  EXP SQRT ABS LOG FLOOR ROUND ISFINITE are Table 1's; the others are
 * extensions the LLM programs need (Table 1 has no erf / sigmoid / rsqrt). */
enum {
  DVM_EXP = 0, DVM_SQRT = 1, DVM_RSQRT = 2, DVM_ABS = 3, DVM_LOG = 4, DVM_ERF = 5,
  DVM_SIGMOID = 6, DVM_NEG = 7, DVM_RECIP = 8, DVM_FLOOR = 9, DVM_ROUND = 10, DVM_TANH = 11,
  DVM_ISFINITE = 12 /* Table 1, IsFinite: the value is 1.0 where x is finite, else 0.0 */
};
/* Binary operators (Table 1: Add Sub Mul Div Min Max Pow).  Pow takes tile operands, like Cmp: an operand
 * that is one value per row makes dvm_encode return DVM_ERR_UNSUPPORTED. */
enum { DVM_ADD = 0, DVM_SUB = 1, DVM_MUL = 2, DVM_DIV = 3, DVM_MIN = 4, DVM_MAX = 5, DVM_POW = 6 };
/* Tensor-scalar operators (Table 1: Adds, Muls). */
enum { DVM_ADDS = 0, DVM_MULS = 1 };
/* Comparisons (Table 1: Cmp): the value is 1.0 where the relation holds, else 0.0. */
enum { DVM_CMP_GT = 0, DVM_CMP_GE = 1, DVM_CMP_LT = 2, DVM_CMP_LE = 3, DVM_CMP_EQ = 4, DVM_CMP_NE = 5 };
/* Row reductions over the last axis, keepdim (Table 1: Sum / Max / Min with N = 1). */
enum { DVM_SUM = 0, DVM_RMAX = 1, DVM_RMIN = 2 };

typedef struct dvm_program dvm_program; /* opaque; owned by the library */

typedef struct {
  int32_t rank;                /* 0 <= rank <= DVM_MAX_RANK */
  int64_t dims[DVM_MAX_RANK];  /* row-major, dense */
} dvm_shape;

/* ------------------------------------------------------------------------
 * Program description: the shape-agnostic "computation graph of basic
 * operators to fuse" (Sec. 3).  Built once, immutable after finalize, shared
 * by every instance.  Each builder call appends one node and returns its
 * value id in *value_id; operands must be earlier value ids.
 * All pointers are host pointers.
 * ---------------------------------------------------------------------- */
int dvm_program_create(dvm_program** out);
void dvm_program_destroy(dvm_program* p); /* NULL is allowed */

/* A global-memory input of the given element type and rank. */
int dvm_program_input(dvm_program* p, int dtype, int rank, int* value_id);
/* Table 1 unary rows (Sqrt Abs Log Exp Round Floor) + extensions. */
int dvm_program_unary(dvm_program* p, int op, int x, int* value_id);
/* Table 1 binary rows; operands broadcast (Table 1, Broadcast). */
int dvm_program_binary(dvm_program* p, int op, int x, int y, int* value_id);
/* Table 1 Adds / Muls with an fp32 immediate. */
int dvm_program_scalar(dvm_program* p, int op, int x, float s, int* value_id);
/* Same, the scalar being runtime argument `param` of dvm_encode (e.g. 1/cols). */
int dvm_program_scalar_param(dvm_program* p, int op, int x, int param, int* value_id);
/* Table 1 Cmp: x `op` y elementwise (operands broadcast), 1.0 / 0.0. */
int dvm_program_compare(dvm_program* p, int op, int x, int y, int* value_id);
/* Table 1 Select: cond != 0 ? x : y elementwise (operands broadcast).  Cmp and Select take tile operands:
 * an operand that is one value per row makes dvm_encode return DVM_ERR_UNSUPPORTED. */
int dvm_program_select(dvm_program* p, int cond, int x, int y, int* value_id);
/* Table 1 Cast: rounds the value to `dtype` (BF16 / F32: nearest even; U8 / I32: toward zero, kept inside the
 * type's range); values stay fp32 in registers. */
int dvm_program_cast(dvm_program* p, int x, int dtype, int* value_id);
/* Table 1 Sum / Max / Min of [M, size, N] over `size` -> [M, 1, N] (the reduced axis stays with size 1).
 * `axis` counts from the end of x's (right-aligned) shape: -1 the last axis (N = 1: threads of a row combine
 * their partial results), -2 the penultimate one (the table's general form), ... down to -DVM_MAX_RANK;
 * a non-negative axis is DVM_ERR_INVALID_ARG.  A reduction over another axis than the last is encoded over
 * views: dvm_encode moves that axis to the end for every operand of the program (shapes and strides alike),
 * so its elements are gathered with the stride the axis has in memory -- correct for every shape, fast only
 * when that stride is small.  A reduction over such an axis that is a RESULT ONLY (nothing in the program reads
 * it, stored as fp32 into a dense output) is encoded differently: the tiles keep their natural shape and
 * combine their rows into the result with atomic operations; dvm_launch first fills that output with the
 * operation's identity (one more small kernel on the stream), and a sum's order of additions is not fixed
 * from run to run (the fp32 result varies in its last bits).  All reductions of one program must name the same axis
 * (dvm_encode: DVM_ERR_UNSUPPORTED otherwise; the streaming fuser, dvm_fuser_reduce_axis, splits such a chain into
 * two meta-kernels on consecutive levels).
 * Length of the reduced axis: up to 8192 elements a row is one tile.  A longer LAST axis is walked in column
 * blocks, in as many passes as the program has reductions that depend on one another (a softmax: maximum, sum
 * of exponentials, quotient; at most 8 passes and 8 per-row values, DVM_ERR_UNSUPPORTED beyond): such a program
 * runs through dvm_launch only, not in a stacked launch.  Another axis than the last that is read back by the
 * program must fit 8192 elements. */
int dvm_program_reduce(dvm_program* p, int op, int x, int axis, int* value_id);
/* The cube operation (Sec. 4.2, matrix operations): a [M,K] x b [K,N], bf16 inputs, fp32 value.
 * Both operands must be program inputs; every matmul of a program shares `a`. */
int dvm_program_matmul(dvm_program* p, int a, int b, int* value_id);
/* Marks value x as an output stored with element type `dtype` (cast on store). */
int dvm_program_output(dvm_program* p, int x, int dtype);
/* Validates the graph.  Required before dvm_encode. */
int dvm_program_finalize(dvm_program* p);
int dvm_program_num_inputs(const dvm_program* p);
int dvm_program_num_outputs(const dvm_program* p);

/* ------------------------------------------------------------------------
 * Per-instance encode (Sec. 4.2: shape tiling, then bytecode encoding).
 * Pure CPU, no CUDA call, no heap allocation; thread-safe on a finalized
 * program.
 *   in_shapes[n_in]    concrete input shapes, in input order
 *   scalars[n_scalars] runtime scalar arguments (may be NULL when n_scalars = 0)
 *   code               caller-owned host buffer of code_capacity bytes, 8-byte aligned
 *   *code_size         receives the encoded size in bytes (also on BUFFER_TOO_SMALL)
 *   out_shapes[n_out]  receives the inferred output shapes (may be NULL)
 * ---------------------------------------------------------------------- */
int dvm_encode(const dvm_program* p, const dvm_shape* in_shapes, int n_in,
               const float* scalars, int n_scalars,
               void* code, size_t code_capacity, size_t* code_size,
               dvm_shape* out_shapes, int n_out);
/* dvm_encode on VIEWS (Table 1, ViewLoad / ViewStore: non-contiguous tiles described by per-dim strides).
 * in_strides[i] (one per input, or in_strides == NULL: all dense) gives the element stride of every dim of
 * in_shapes[i]: element (i_0 .. i_{r-1}) of input i lies at tensors[i] + sum_k i_k * stride[k] elements, so
 * the tensor pointer passed at launch is the address of the view's first element.  out_strides[o] (one per
 * output, or NULL) does the same for output o over the dims out_shapes[o] reports.  Strides of dims of size
 * 1 are ignored; a stride of 0 on an input dim repeats the element (an expanded view).
 *  - DVM_ERR_INVALID_ARG: a negative stride; an output view that addresses an element twice (a zero stride,
 *    or dims that overlap).
 *  - DVM_ERR_UNSUPPORTED: more than three outer dims left after adjacent dims that are dense in every
 *    operand were merged; a program with a matmul.
 * Cost: a view whose last dim is adjacent in memory (stride 1: slices, permuted outer dims, padded rows) is
 * copied row by row as byte ranges, like a dense tensor.  A view whose last dim is strided (a transpose that
 * moves the last dim, a column slice with a step, a last dim expanded with stride 0) is gathered / scattered
 * element by element: correct, but every element costs a 32-byte memory sector.
 * Everything else as dvm_encode. */
typedef struct {
  int64_t stride[DVM_MAX_RANK]; /* elements; entry k belongs to dim k of the shape */
} dvm_strides;
int dvm_encode_strided(const dvm_program* p, const dvm_shape* in_shapes, const dvm_strides* in_strides, int n_in,
                       const float* scalars, int n_scalars, const dvm_strides* out_strides,
                       void* code, size_t code_capacity, size_t* code_size,
                       dvm_shape* out_shapes, int n_out);
/* Measurement helper: calls the encoder `reps` times on one instance (in_strides may be NULL: dense inputs) and
 * writes the duration of every call, in nanoseconds of the steady clock, to ns_out[0 .. reps).  The clock is read
 * inside the library, so the figures hold the encoder alone -- no binding, no interpreter of the caller's
 * language.  `code` / `code_capacity`: a caller-owned buffer as for dvm_encode.  Host pointers throughout. */
int dvm_time_encode(const dvm_program* p, const dvm_shape* in_shapes, const dvm_strides* in_strides, int n_in,
                    const float* scalars, int n_scalars, void* code, size_t code_capacity, int reps, int64_t* ns_out);
/* dvm_encode for n independent instances in one call -- the stacked-fusion case (Sec. 5.1), where every
 * program of a launch is re-encoded per launch.  All arrays are host memory of length n, except
 * in_shapes / scalars, which concatenate the instances' arguments (instance i consumes n_in[i] shapes and
 * n_scalars[i] scalars).  codes[i] is a caller-owned 8-byte aligned buffer of caps[i] bytes; sizes[i]
 * receives the encoded size.  Output shapes are not returned (encode the instance alone to get them).
 * Stops at the first instance that fails and returns its status, *failed (may be NULL) = its index. */
int dvm_encode_batch(int n, const dvm_program* const* programs, const dvm_shape* in_shapes, const int* n_in,
                     const float* scalars, const int* n_scalars, void* const* codes, const size_t* caps,
                     size_t* sizes, int* failed);
/* Upper bound of the encoded size, in bytes, for any shape. */
size_t dvm_code_max_size(const dvm_program* p);

/* Number of parallel units N the tiling cost model balances for (Sec. 4.2: cost
 * = ceil(#tiles / N) * (tile + overhead)).  Default 444 (148 SMs x 3); the encoder scales it to the
 * CTAs that are actually resident per SM for the instance (at most 2).
 * n <= 0 restores the default.  Per calling thread (the setting of one thread does not reach the encodes of another). */
void dvm_set_num_cores(int n);
int dvm_get_num_cores(void);
/* Elements of a tile register that one thread holds (the analogue of the paper's tile size
 * limit T_max = M / n_max): 16, 24 or 32.  0 (default) lets the cost model choose per instance (24 only for
 * programs of the basic instruction set on dense tensors: it exists for dvm_launch alone, a stacked launch of
 * a 24-element program returns DVM_ERR_UNSUPPORTED).
 * Programs stacked into one launch must all use the same value, so callers of
 * dvm_launch_stacked fix it before encoding.  Per calling thread (the setting of one thread does not reach the encodes of another). */
void dvm_set_elems_per_thread(int v);
int dvm_get_elems_per_thread(void);
/* Resident CTAs per SM every encoded geometry has to leave room for: 2, or 0 (default) for no constraint.
 * A stacked launch sizes every CTA's local memory for its largest program, so ONE program whose tile slots
 * exceed half an SM's shared memory leaves the whole launch with one CTA per SM.  With 2, the encoder
 * takes the best geometry among those whose slots fit twice per SM (e.g. two column blocks per row, whose
 * row-vector operands are then half as long); a program no geometry of which fits keeps its unconstrained
 * best.  Callers of dvm_launch_stacked set it before encoding.  Per calling thread (the setting of one thread does not reach the encodes of another).
 * n = 3: as 2, for stacked launches that run with ONE tile slot per CTA (dvm_set_stacked_one_slot): a geometry has
 * to leave room for two CTAs that hold one slot each, so tiles may be twice as large. */
void dvm_set_min_resident_ctas(int n);
/* Stacked launches of this process (dvm_launch_stacked, and the flushes of the streaming fuser) run with one tile
 * slot per CTA when `on` != 0: a tile's loads start when the CTA's previous tile is done (no load-ahead inside a
 * CTA; the SM's other CTA computes meanwhile), every program on one level of the variant with level waits.  For
 * programs encoded with dvm_set_min_resident_ctas(3); programs whose single slot does not fit twice leave the launch
 * with one CTA per SM.  Default off. */
void dvm_set_stacked_one_slot(int on);
int dvm_get_min_resident_ctas(void);
/* One-program launches of the basic instruction set run on a lean variant of the interpreter (Algorithm 2 from
 * linked code: a shorter instruction stream per tile).  0 sends every launch of the process to the general
 * interpreter instead, 2 also sends stacked launches to the lean one (for comparisons; measured slower).
 * Default 1.  Both interpreters run the same bytecode and give results inside the same tolerances. */
void dvm_set_lean_kernel(int on);

/* Which build of the interpreter the calling thread's last vector launch ran on (for tests and tools): out =
 * { elements per thread, 1 for the 32 KB parameter block, 1 for one program per launch, extension level, 1 with
 *   level waits, lean, 1 with the heavy unary functions, resident CTAs per SM it is compiled for }.  lean: 0 the
 * general interpreter; 1 the lean one with every path; 2 its build for phased programs; 3 for two tile slots;
 * 4 ... and dense loads (no row-by-row copies, per-row scalar inputs, outer dims); 5 ... and aligned operands (no
 * realignment of reads); 6 two slots and aligned operands with row-by-row copies; 7 as 5 for rows that fill the
 * tile's slots exactly (no slot masks); 8 as 6 for such rows; 9 aligned programs with one tile slot.  DVM_ERR_INVALID_ARG before the thread's first launch. */
int dvm_last_launch_variant(int out[8]);

/* Matmul launches (Sec. 4.2, matrix operations): the tiles of a last, partial wave are shared along k -- a small
 * wave gives each tile up to four CTAs (or CTA pairs), a larger one is cut into equal ranges of its k blocks over
 * all of them -- whenever the k blocks saved outweigh the exchange (decided per launch from its shape).  The
 * shares meet in a library-owned fp32 workspace (one per device and stream, 26 MB, allocated by the first launch
 * that needs it; launches into a stream that is being captured run unsplit) and are added in
 * a fixed order, so results are deterministic.  They differ from the unsplit result by fp32 rounding of the
 * partial sums.  on = 0 switches the split off.  Default 1. */
void dvm_set_matmul_tail_split(int on);

/* The tail split a matmul launch of `tiles` output tiles with `k_blocks` blocks of 64 along k would use on `units`
 * CTAs (ctas_per_unit = 1) or CTA pairs (2).  Returns 0 when such a launch does not split, 1 when it does, and then
 * out = { first tile of the last wave, its tiles r, most parts of a tile, k blocks per unit W, pitch P of the tiles
 * on the line of k blocks, units that take part }: tile a of the wave lies at blocks [a P, a P + k_blocks) of the
 * line, unit c takes [c W, (c + 1) W), the unit holding a tile's first block owns it.  Host only (the arithmetic
 * of dvm_launch, for tests and tools). */
int dvm_matmul_tail_plan(int64_t tiles, int units, int k_blocks, int ctas_per_unit, int32_t out[6]);

/* Matmul launches on CTA pairs: two CTAs of a cluster compute a tile of 256 output rows with one tcgen05
 * cta_group::2 instruction stream, each loading its own rows of A and half of the B tile (a third less
 * shared-memory traffic per flop).  mode = 0: never; 1 (default): where the launch's shape favours it; 2: wherever
 * the output has at least two blocks of 128 rows.  Results are those of the single-CTA kernel bit for bit (the
 * same instruction shape along k). */
void dvm_set_matmul_cta_pairs(int mode);

/* The paper's tile-size rule for a flat vector operator (Sec. 4.2,
 * hardware_align_div): among tile sizes t in [1, min(total, t_max)] take the
 * one minimising ceil(ceil(total / t) / n_cores) * (t + overhead) (ties: the
 * larger t), then round it up to a multiple of `align` elements without
 * exceeding t_max.  Outputs (each may be NULL): the min-cost tile, the rounded
 * tile, the tile count and tail size for the min-cost tile.  Host only. */
int dvm_hardware_align_div(int64_t total, int n_cores, int64_t align, int64_t t_max,
                           int64_t overhead, int64_t* min_cost_tile, int64_t* rounded_tile,
                           int64_t* n_tiles, int64_t* tail);

/* Algorithm 2's tile range of core `id`: m = ceil(M / N), [m*id, min(M, m*(id+1))). */
int dvm_vm_tile_range(int64_t n_tiles, int n_cores, int id, int64_t* begin, int64_t* end);

/* ------------------------------------------------------------------------
 * Launch (Sec. 4.3, Algorithm 2).  Asynchronous on `cuda_stream` (a
 * cudaStream_t passed as void*; NULL = default stream).  `code` is a host
 * pointer; it is copied into the launch, so the caller may reuse it when the
 * call returns.  tensors[n_tensors] are DEVICE pointers, inputs then outputs,
 * caller-owned, element-aligned; they must stay valid until the stream has run
 * the kernel.  Zero-size instances launch nothing.
 * ---------------------------------------------------------------------- */
int dvm_launch(const void* code, size_t code_size, void* const* tensors, int n_tensors,
               void* cuda_stream);

/* Stacking-based fusion (Sec. 5.1): n_programs independent vector meta-kernels
 * run as ONE kernel; their tiles are claimed from one work queue, spread over
 * SMs (spatial) and run back to back on each SM (temporal).
 * codes[i] / code_sizes[i] / tensors[i] / n_tensors[i] as for dvm_launch.  All programs must have
 * been encoded with the same elements-per-thread setting (DVM_ERR_INVALID_ARG otherwise).
 * Limits (DVM_ERR_TOO_LARGE beyond): 256 programs, and the programs travel together in the 32 KB
 * kernel-parameter block: the sum of their code sizes plus 8 bytes per program must stay within 32000 bytes
 * (about 130 programs of three tensors each). */
int dvm_launch_stacked(int n_programs, const void* const* codes, const size_t* code_sizes,
                       void* const* const* tensors, const int* n_tensors, void* cuda_stream);

/* Temporal stacking of DEPENDENT meta-kernels (Sec. 5.1: stacking in time puts tiles of different operators
 * one after the other on a core, so it also covers operators that depend on one another).  As dvm_launch_stacked,
 * plus level[n_programs] (host): a program may read tensors that programs of LOWER levels of the same call
 * write; programs of one level must be independent of one another.  Levels must be non-decreasing in i
 * (DVM_ERR_INVALID_ARG otherwise): the work queue hands tiles out in that order.  Inside the kernel a tile
 * of level L starts its loads only when every tile of the lower levels has been counted complete (stores
 * fenced device-wide); that wait is bounded (about 2 s), after which the kernel records
 * DVM_ERR_DEVICE_TIMEOUT for dvm_last_device_status and returns.  The grid never exceeds the number of
 * CTAs the device keeps resident, so every tile a waiting CTA depends on is held by a running CTA. */
int dvm_launch_stacked_levels(int n_programs, const void* const* codes, const size_t* code_sizes,
                              void* const* const* tensors, const int* n_tensors, const int* level,
                              void* cuda_stream);

/* The stacked launch for callers that must not allocate device memory.  (The paper has no counterpart:
 * this entry point exists for deployment, not for the method.)
 *
 * dvm_launch_stacked keeps its work-queue counters in a small device buffer that the library cudaMalloc's
 * the first time it is used on a device.  Callers that run inside a memory pool owning the whole device,
 * serving loops that cannot afford the implicit synchronisation of a first-use cudaMalloc, and sandboxes
 * that forbid the allocator cannot use it.  This variant runs the same kernel with the counters in a fixed
 * 256-byte array inside the library image (every GPU that loads the library holds it until the process
 * exits) and calls neither cudaMalloc nor cudaFree nor any allocating routine.
 *  - Arguments, tensor ownership and the result are those of dvm_launch_stacked.
 *  - Limits: at most DVM_NOALLOC_MAX_PROGRAMS programs and DVM_NOALLOC_MAX_TILES tiles per call;
 *    larger requests return DVM_ERR_TOO_LARGE.
 *  - The first call on a device resolves the array's device address (cudaGetSymbolAddress) and reads the
 *    SM count; make that first call before any stream capture.
 *  - Every call shares the array, and the array keeps the last call's contents: each call clears it on
 *    `cuda_stream` before its kernel.  Two calls whose kernels overlap on the GPU (different streams) race
 *    on it -- serialise them.
 *  - Device-side status is not reported for this variant (the bytecode is verified on the host first). */
#define DVM_NOALLOC_MAX_PROGRAMS 256
#define DVM_NOALLOC_MAX_TILES 0x7fffffffull
int dvm_launch_stacked_noalloc(int n_programs, const void* const* codes, const size_t* code_sizes,
                               void* const* const* tensors, const int* n_tensors, void* cuda_stream);

/* End-to-end convenience for HOST tensors: copies the inputs to device staging
 * memory the caller provides (`staging`, device pointer, staging_bytes >= sum of
 * all tensor sizes rounded up to 256 B each), launches, copies the outputs back
 * and synchronises the stream.  host_tensors[i] has tensor_bytes[i] bytes;
 * pinned host memory makes the copies asynchronous.
 * When every tensor of a vector program either follows the tiles (a dense operand) or is a row vector, and the
 * tensors total 64 MB or more, the call pipelines: the tiles run in chunks (Algorithm 2's tile ranges), each chunk
 * copying its input rows in, executing and copying its output rows out on one of three library-owned streams, so
 * that copies in both directions overlap execution.  The result is the same; the call still returns after everything
 * has finished on `cuda_stream`. */
int dvm_run_host(const void* code, size_t code_size, void* const* host_tensors,
                 const size_t* tensor_bytes, int n_tensors, void* staging, size_t staging_bytes,
                 void* cuda_stream);

/* ------------------------------------------------------------------------
 * Support
 * ---------------------------------------------------------------------- */
/* Host-side validation of a bytecode program (every instruction id, length,
 * register, operand and slot index, table sizes).  dvm_launch runs it too. */
int dvm_verify(const void* code, size_t code_size);
/* Readable dump (the paper's Fig. 5 prints one: tile count, per-core tiles,
 * kernel type, one line per operation).  Returns DVM_ERR_BUFFER_TOO_SMALL if
 * `cap` is too small; the text is always NUL-terminated when cap > 0. */
int dvm_disassemble(const void* code, size_t code_size, char* buf, size_t cap);
/* Header fields of an encoded program (each output may be NULL). */
int dvm_code_info(const void* code, size_t code_size, int* kernel_type, int64_t* n_tiles,
                  int* code_body_bytes, int* threads_per_row, int* vector_width, int* n_tile_regs);
/* The bytes of every tensor slot that a launch of `code` reads or writes, counted from the pointer given at launch
 * (inputs first, then outputs): bytes_needed[i] = 1 + the largest byte offset the program addresses in slot i, 0 for
 * a slot nothing addresses or an empty program.  Host only.  (Tile loads fetch whole 16-byte units: a launch may
 * READ up to 15 bytes on either side of an input's range, inside the same 16-byte aligned units.) */
int dvm_tensor_extents(const void* code, size_t code_size, int64_t* bytes_needed, int n_tensors);
/* dvm_launch behind a bounds check: DVM_ERR_BUFFER_TOO_SMALL when some tensor_bytes[i] (host array) is below what
 * dvm_tensor_extents reports, before anything is launched.
 * Debug mode: with the environment variable DVM_DEBUG=1 every launch of this library (checked or not) runs on the
 * general interpreter with its device-side checks on (register, operand and tensor-slot indices and instruction
 * lengths of every decoded instruction; a failed check sets the status word instead of touching memory),
 * synchronises the stream and returns the device status (DVM_ERR_DEVICE_*) as its own. */
int dvm_launch_checked(const void* code, size_t code_size, void* const* tensors, const size_t* tensor_bytes,
                       int n_tensors, void* cuda_stream);
/* Self-test of the bounded device-side waits (no counterpart in the paper): launches one CTA that waits on
 * an mbarrier nobody completes, with the very wait routine of the interpreter (which = 0) or of the matmul
 * kernel (which = 1), or on a tile counter nobody advances with the level wait of dvm_launch_stacked_levels
 * (which = 2).  The wait gives up after its limit (about 2 s), the kernel sets the status word and
 * returns: dvm_last_device_status then reports DVM_ERR_DEVICE_TIMEOUT and the context stays usable. */
int dvm_selftest_bounded_wait(int which, void* cuda_stream);
/* Synchronises `cuda_stream`, then reads and clears the device status word of
 * the current device: *status is DVM_OK or a DVM_ERR_DEVICE_* code. */
int dvm_last_device_status(void* cuda_stream, int* status);
/* The cudaError_t (as int) of the last failed CUDA call on this thread. */
int dvm_last_cuda_error(void);
/* Number of kernels this library has launched in this process. */
int64_t dvm_launch_count(void);
const char* dvm_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* DVM_H_ */
