/* libdvm -- the streaming runtime operator fuser (Sec. 5.2, "Fusion on Static/Dynamic Graphs",
 * dynamic computation graphs): operators arrive one at a time while a dynamic model runs, are added to a
 * buffer, fusion decisions are made immediately, and the fused operators are flushed to the operator
 * compiler (dvm_encode) and executed (dvm_launch / dvm_launch_stacked) when a flush condition occurs.
 *
 * Fusion rules (Sec. 5.1):
 *  - pattern-based, vector-vector: an arriving operator joins the open group that produced its operands
 *    when the iterations merge, i.e. when the group with the operator still encodes as ONE meta-kernel for
 *    the concrete shapes (the test is a trial dvm_encode: a few microseconds);
 *  - stacking-based: groups that do not depend on one another are launched together as one stacked kernel
 *    (spatial stacking); a group that consumes another group's result joins the same kernel one level later
 *    (temporal stacking of dependent operators, dvm_launch_stacked_levels), so that a flush of short levels
 *    is ONE launch.  With temporal stacking switched off, when a level has more than 1024 tiles (4 M
 *    elements: the host is then far ahead of the device and kernel boundaries cost nothing extra), or when
 *    the groups do not fit one launch, each level is its own launch on the stream.
 * Flush conditions: dvm_fuser_flush (a result has to go back to the host, a synchronisation point), or the
 * operator buffer is full.  A value whose last reference the framework dropped before the flush
 * (dvm_fuser_release) and that no other group reads is never stored to global memory: that store is the
 * traffic fusion removes.
 *
 * Conventions as in dvm.h: every call returns DVM_OK or a negative DVM_ERR_*; host pointers unless stated;
 * tensors are dense row-major device memory owned by the caller and must stay valid until the flush that
 * runs their operators has been issued and the stream has executed it.  Not thread-safe.
 */
#ifndef DVM_FUSER_H_
#define DVM_FUSER_H_

#include "dvm.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dvm_fuser dvm_fuser; /* opaque; owned by the library */

#define DVM_FUSER_MAX_OPS 256 /* operators buffered between two flushes; one more flushes first */

/* cuda_stream: the stream every launch of this fuser is issued on (cudaStream_t as void*, NULL = default). */
int dvm_fuser_create(dvm_fuser** out, void* cuda_stream);
void dvm_fuser_destroy(dvm_fuser* f); /* pending operators are dropped, not run; NULL is allowed */

/* Temporal stacking of dependent groups in one launch: on (non-zero, the default) or off. */
int dvm_fuser_set_temporal_stacking(dvm_fuser* f, int enabled);

/* A tensor that already exists in device memory (a graph input, a parameter): *value names it. */
int dvm_fuser_tensor(dvm_fuser* f, int dtype, const dvm_shape* shape, void* device_ptr, int* value);

/* Operators (Table 1 semantics, as the dvm_program_* builders).  `out_ptr` is the device buffer the framework
 * allocated for the result (element type out_dtype); *out_shape (may be NULL) receives the result's shape,
 * *value its id.  Nothing runs before a flush. */
int dvm_fuser_unary(dvm_fuser* f, int op, int x, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);
int dvm_fuser_binary(dvm_fuser* f, int op, int x, int y, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);
int dvm_fuser_scalar(dvm_fuser* f, int op, int x, float s, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);
int dvm_fuser_reduce(dvm_fuser* f, int op, int x, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);
/* The same over another axis (axis < 0, counted from the end; -1 is dvm_fuser_reduce).  One meta-kernel reduces over
 * one axis: an operator that reduces over a second axis, or that reads across the first one's result in another
 * direction, opens the next group, one level up -- a chain with two reduced axes runs as two stacked levels. */
int dvm_fuser_reduce_axis(dvm_fuser* f, int op, int x, int axis, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);
/* Table 1 Cmp, Select (cond != 0 ? x : y), Cast (the value rounded to `dtype`), and the cube operation a [M,K] x b [K,N]
 * (Sec. 4.2; bf16 operands that lie in memory).  A matmul starts a group of its own; the vector operators that
 * arrive behind it join that group as its epilogue while the group still encodes as one matmul meta-kernel --
 * cube-vector fusion (Sec. 5.1) on arrival.  out_dtype may be DVM_U8 / DVM_I32 (a comparison stored as 0 / 1, a cast);
 * a value of an integer type can be read by later operators of its own group only (tensors in memory are F32 / BF16). */
int dvm_fuser_compare(dvm_fuser* f, int op, int x, int y, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);
int dvm_fuser_select(dvm_fuser* f, int cond, int x, int y, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);
int dvm_fuser_cast(dvm_fuser* f, int x, int dtype, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);
int dvm_fuser_matmul(dvm_fuser* f, int a, int b, int out_dtype, void* out_ptr, dvm_shape* out_shape, int* value);

/* The framework dropped its last reference to `value`: if it is still pending and only its own group reads
 * it, it will not be stored. */
int dvm_fuser_release(dvm_fuser* f, int value);

/* Flush: every buffered operator is compiled and launched (asynchronously, on the fuser's stream); afterwards
 * every value that was not released lies in its buffer once the stream has run. */
int dvm_fuser_flush(dvm_fuser* f);

/* What is buffered right now (each may be NULL): operators not yet flushed, and the fused groups they form. */
int dvm_fuser_pending(const dvm_fuser* f, int* n_ops, int* n_groups);

/* Counters since creation (each may be NULL): operators received, fused groups (meta-kernels) built, kernel
 * launches issued, result stores elided. */
int dvm_fuser_stats(const dvm_fuser* f, int64_t* n_ops, int64_t* n_groups, int64_t* n_launches, int64_t* n_stores_elided);

#ifdef __cplusplus
}
#endif
#endif /* DVM_FUSER_H_ */
