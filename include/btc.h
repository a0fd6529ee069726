/*
 * btc.h -- C interface of the B200 tensor-contraction library.
 *
 * One operation:   D := alpha * op(A) * op(B) + beta * op(C)
 *
 * A, B, C, D are dense tensors in a general strided layout (an element with indices
 * i_0..i_{n-1} lives at base + sum_k i_k * stride_k; Glossary, "Strided layout").  Every mode
 * carries an index label.  Labels shared by A and B only are contracted (summed); labels shared
 * by one input and D are free and may appear in D in any order; labels shared by A, B and D are
 * Hadamard (batch) labels (Sec. "Operations", Cases 1-2, Eq. (case1), Eq. (case2)).  A label may
 * occur several times inside A or inside B (Case 3; such a tensor equals one with a single mode
 * whose stride is the sum of the strides, Note 6).  op() optionally conjugates complex operands.
 *
 * The object model follows Sec. "Interface Components": a library handle, tensor descriptors
 * that hold no data pointer, an operation descriptor that is validated and planned once, and an
 * execute call that takes only data pointers, scalars and an executor (here: a CUDA stream).
 * Every function returns an integer error code (0 = success; the other values are not part of
 * the contract, use btc_explain_error); outputs are returned through pointers; destroy functions
 * take the address of the handle and null it (Sec. "Error Handling").
 *
 * Threads: objects are immutable after creation except through btc_set_attr; executing one
 * contraction object from several host threads is allowed when each call has its own workspace.
 *
 * complex64 operations of at least about 2 GFLOP run as a real fp32 contraction on the tensor cores: the
 * smaller input is first expanded into the workspace (16 bytes per element; counted in
 * btc_contraction_workspace_size).  A call whose workspace has no room for that (or none at all, or the
 * library's static scratch when it is too small) runs the complex kernels instead, with the same result
 * within the tolerance.  The kernel, variant, tile and grid attributes describe the fp32 contraction.
 *
 * Environment: BTC_LOG (any value) prints every contraction's plan to stderr when it is created,
 * and a note when a problem of more than 1 GFLOP lands on the per-element kernel.
 */
#ifndef BTC_H_
#define BTC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int btc_error_t;

enum {
    BTC_SUCCESS = 0,
    BTC_ERR_INVALID_ARGUMENT = 1,    /* NULL where a value is required, bad rank, bad enum      */
    BTC_ERR_INVALID_EXTENT = 2,      /* an extent < 1 (extents are positive integers)           */
    BTC_ERR_EXTENT_MISMATCH = 3,     /* one label with two extents (test list item 26)          */
    BTC_ERR_C_D_MISMATCH = 4,        /* C's rank, extents, strides or labels differ from D's    */
    BTC_ERR_D_ALIASING = 5,          /* two index tuples of D address one element (item 28)     */
    BTC_ERR_LABEL_ONLY_IN_D = 6,     /* a label of D in neither A nor B (Eq. (FreeD), Case 5)   */
    BTC_ERR_NOT_SUPPORTED = 7,       /* unsupported mix of element types, label repeated inside D */
    BTC_ERR_WORKSPACE_TOO_SMALL = 8,
    BTC_ERR_MISALIGNED = 9,          /* a data pointer not aligned to its element size          */
    BTC_ERR_CUDA = 10,               /* a CUDA runtime call failed                              */
    BTC_ERR_DEVICE_TIMEOUT = 11,     /* a bounded device-side wait expired                      */
    BTC_ERR_OUT_OF_MEMORY = 12,
    BTC_ERR_SCRATCH_LIMIT = 13       /* needs more than the built-in scratch array holds        */
};

/* Element types.  Complex values are (re, im) pairs of the stated part width. */
typedef enum {
    BTC_F32 = 0,
    BTC_F64 = 1,
    BTC_C32 = 2, /* 2 x float  (8 bytes)  */
    BTC_C64 = 3  /* 2 x double (16 bytes) */
} btc_dtype_t;

typedef struct btc_handle_s *btc_handle_t;            /* Sec. "The Library Handle"            */
typedef struct btc_tensor_info_s *btc_tensor_info_t;  /* Sec. "Tensor Descriptors"            */
typedef struct btc_contraction_s *btc_contraction_t;  /* Sec. "Tensor Operation Descriptors"  */
typedef struct btc_status_s *btc_status_t;            /* Sec. "Status Objects"                */

#define BTC_MAX_RANK 32
#define BTC_MAX_LABELS 64

/* Library handle (Sec. "The Library Handle").  Binds the CUDA device that is current on the
 * calling thread; every object made from it lives on that device.  Host memory only. */
btc_error_t btc_create_handle(btc_handle_t *out);
btc_error_t btc_destroy_handle(btc_handle_t *handle); /* *handle becomes NULL */

/* Tensor descriptor (Sec. "Tensor Descriptors"): rank, extents, strides, element type; no data.
 *   rank      0..BTC_MAX_RANK; rank 0 is a scalar (Note 2, Note 4)
 *   extents   host array of `rank` entries, each >= 1; may be NULL iff rank == 0
 *   strides   host array of `rank` entries in ELEMENTS, signed, zero allowed; NULL means dense
 *             column-major (stride_0 = 1, stride_k = prod_{l<k} extent_l; Glossary)
 * The arrays are copied.  Errors: INVALID_ARGUMENT, INVALID_EXTENT. */
btc_error_t btc_create_tensor_info(btc_handle_t handle, btc_dtype_t dtype, int32_t rank,
                                   const int64_t *extents, const int64_t *strides,
                                   btc_tensor_info_t *out);
btc_error_t btc_destroy_tensor_info(btc_tensor_info_t *info);

/* Operation descriptor (Sec. "Tensor Operation Descriptors"; the checks of Sec. "Algorithm
 * Structure", first paragraph; label classification of Sec. "Operations").
 *   A, B, D     tensor descriptors (copied; they may be destroyed or reused afterwards)
 *   C           descriptor of C, or NULL when the operation never reads C (then beta must be 0
 *               at every execute).  C must have D's rank, extents, strides and label order
 *               (Note 5).
 *   labelsX     host array, one int64 label per mode of X (any values); NULL iff rank 0
 *   conjX       non-zero: op(X) = element-wise complex conjugate; ignored for real types
 *   alpha,beta  host scalars of D's element type stored as the defaults of the operation;
 *               NULL means alpha = 1, beta = 0
 * Element types (Sec. "Challenge: Datatypes"): normally all four tensors share one type.  Real and
 * complex tensors of one part width may be mixed (a real operand counts as complex with zero
 * imaginary parts) as long as D is complex whenever A, B or C is.  One real and one complex input
 * with a complex C (or none), real alpha and beta and no conjugation of the complex tensors run on
 * the tiled kernels (the complex tensors are read as real ones with one more mode); other mixes run
 * on the per-element kernel (exact, not fast).  32- and 64-bit parts cannot be mixed (NOT_SUPPORTED).
 * All validation and planning (label classes, mode fusion, kernel and tile choice, device-side
 * offset tables) happens here; the call may allocate device memory and copy small tables with
 * the default stream.  Errors: INVALID_ARGUMENT, EXTENT_MISMATCH, C_D_MISMATCH, D_ALIASING,
 * LABEL_ONLY_IN_D, NOT_SUPPORTED, OUT_OF_MEMORY, CUDA. */
btc_error_t btc_create_contraction(btc_handle_t handle,
                                   btc_tensor_info_t A, const int64_t *labelsA, int conjA,
                                   btc_tensor_info_t B, const int64_t *labelsB, int conjB,
                                   btc_tensor_info_t C, const int64_t *labelsC, int conjC,
                                   btc_tensor_info_t D, const int64_t *labelsD,
                                   const void *alpha, const void *beta,
                                   btc_contraction_t *out);
btc_error_t btc_destroy_contraction(btc_contraction_t *op);

/* Bytes of device workspace btc_execute needs for this operation (0 for most plans; split-K
 * plans keep their partial sums there, Case 4 plans the inputs summed over their isolated
 * labels).  Alignment required: 256 bytes. */
btc_error_t btc_contraction_workspace_size(btc_contraction_t op, size_t *bytes);

/* Key-value access on an operation (Sec. "Virtual Key-Value Stores").  Values are host memory. */
enum {
    BTC_ATTR_KERNEL = 1,      /* int32, read/write: BTC_KERNEL_* (write re-plans)              */
    BTC_ATTR_SPLIT_K = 2,     /* int32, read/write: number of K slices (>= 1)                  */
    BTC_ATTR_TILE = 3,        /* int32[3], read: CTA tile extents M, N, K                      */
    BTC_ATTR_GROUPS = 4,      /* int64[4], read: batch, M, N, K sizes after classification     */
    BTC_ATTR_GRID = 5,        /* int32[3], read: launch grid                                   */
    BTC_ATTR_NUM_MODES = 6,   /* int32[4], read: modes per class after fusion (batch, M, N, K) */
    BTC_ATTR_SWAPPED = 7,     /* int32, read: 1 when A and B exchanged roles                   */
    BTC_ATTR_VARIANT = 9,     /* int32, read/write: index of the tile variant of the tiled
                                 kernel for this element type (-1 on write = choose).  A variant
                                 the operation cannot use (a bulk-tensor-copy variant whose M-side
                                 tiles are no boxes of the operand) is replaced by its nearest
                                 equivalent; read back what was planned                       */
    BTC_ATTR_DEVICE_ERROR = 8,/* int32, read: 0, or which bounded device-side wait gave up in an
                                 earlier execute of this operation (its D is then incomplete, and
                                 a split-K result is not written at all); reading waits for the
                                 device.  The word is sticky: write 0 to clear it.  btc_execute
                                 cannot report it (it never waits for the device): callers that
                                 need to know poll this attribute after synchronising;
                                 btc_execute_host returns BTC_ERR_DEVICE_TIMEOUT itself           */
    BTC_ATTR_POLL_LIMIT = 13, /* int32 >= 0, write: polls after which a device-side wait gives up
                                 (default 4194304).  For tests of the failure path: with a limit of 0
                                 every wait of the tiled kernels gives up at once, the kernels
                                 return without writing D, and the error word tells; nothing faults
                                 or hangs                                                          */
    BTC_ATTR_COMPUTE_PRECISION = 12, /* int32, read/write (write re-plans): BTC_PRECISION_* -- the compute
                                 precision an operation may ask for (Sec. "Tensor Operation Descriptors").  DEFAULT:
                                 fp32 products are formed from three TF32 tensor-core products (error of a
                                 product <= 2^-22 |a||b|, fp32 accumulation); STRICT: fp32 operations run on
                                 the FMA pipe in IEEE fp32 (about a third of the speed); FP64_SUMS: fp32 /
                                 complex64 storage, products and sums kept in fp64 and rounded once to the
                                 element type (runs the per-element kernel: exact but slow).  No effect on
                                 fp64 and complex128 (always IEEE fp64); STRICT is NOT_SUPPORTED for complex64 */
    BTC_ATTR_BATCH_HINT = 11, /* int32 >= 1, read/write (write re-plans): how many pointer-array entries
                                 btc_execute_batched will usually be given.  Tile variant and split-K
                                 are then chosen for that many entries in flight (no split-K when the
                                 array alone fills the GPU); any count still works with any hint    */
    BTC_ATTR_PRE_REDUCE = 10  /* int32.  Case 4 of Sec. "Operations": labels that occur in one input
                                 only are summed over before the contraction.  Write 1 (default):
                                 a separate bandwidth-bound kernel forms the summed input in the
                                 workspace and the contraction runs on it; write 0: the isolated
                                 labels are summed inside the generic kernel.  Read: bit 0 / bit 1
                                 set when A / B is summed first in the current plan             */
};
enum { BTC_PRECISION_DEFAULT = 0, BTC_PRECISION_STRICT = 1, BTC_PRECISION_FP64_SUMS = 2 };
enum {
    BTC_KERNEL_AUTO = 0,
    BTC_KERNEL_GENERIC = 1,   /* one thread per element of D, any legal input                  */
    BTC_KERNEL_TILED = 2      /* shared-memory tiled contraction kernel                        */
};
btc_error_t btc_set_attr(btc_contraction_t op, int32_t key, const void *value, size_t len);
btc_error_t btc_get_attr(btc_contraction_t op, int32_t key, void *value, size_t len, size_t *needed);

/* Execute (Sec. "Execution"): enqueue the operation on a stream and return.
 *   cuda_stream  a cudaStream_t passed as void*; NULL is the default stream (the "default
 *                executor" of Sec. "Executors")
 *   alpha, beta  HOST pointers to scalars of D's element type, or NULL for the stored defaults.
 *                beta == 0: C is not read (may be NULL); alpha == 0: A and B are not read.
 *   A, B, C, D   DEVICE pointers to the logical element (0,...,0) of each tensor, aligned to the
 *                element size.  C == D (same pointer) is the in-place update.  Any other overlap
 *                of D with A, B or C is undefined.  The caller owns all buffers.
 *   workspace    DEVICE pointer, 256-byte aligned, at least btc_contraction_workspace_size bytes
 *                (may be NULL when that size is 0)
 *   status       NULL, or receives a new status object describing the launch (destroy it)
 * The call never allocates device memory and never synchronises.  Errors: INVALID_ARGUMENT,
 * MISALIGNED, WORKSPACE_TOO_SMALL, CUDA (launch failure). */
btc_error_t btc_execute(btc_contraction_t op, void *cuda_stream,
                        const void *alpha, const void *A, const void *B,
                        const void *beta, const void *C, void *D,
                        void *workspace, size_t workspace_bytes,
                        btc_status_t *status);

/* Convenience for callers whose buffers live in HOST memory: copies A, B (and C when beta != 0)
 * to device buffers it allocates, executes, copies D back, and synchronises the stream.  Large
 * operations run in slabs: the larger input is cut along the label with its largest stride and slab
 * i + 1 is copied (on a stream of the library's own) while slab i is contracted, so that the transfer
 * hides the arithmetic; a contracted label's slabs accumulate into D, which changes the order of the
 * sum, not its value beyond rounding.  The device buffers of this path stay with the operation object
 * until it is destroyed or re-planned; calls on one operation object must not overlap in time.
 * Pinned host memory is what lets the copies overlap.
 * Pointers address logical element (0,...,0) of host tensors laid out as the descriptors say;
 * each tensor's whole strided span is transferred.  Errors as btc_execute plus OUT_OF_MEMORY, and
 * DEVICE_TIMEOUT when a bounded device-side wait gave up (D is then incomplete). */
btc_error_t btc_execute_host(btc_contraction_t op, void *cuda_stream,
                             const void *alpha, const void *A, const void *B,
                             const void *beta, const void *C, void *D);

/* Batched execution with pointer arrays (Sec. "Tensor Descriptors": descriptors hold no data pointer
 * so that one description serves many tensors, batched operations among them).
 * Executes the operation `count` times, entry i on A[i], B[i], C[i], D[i]; alpha and beta are shared.
 *   A, B, C, D   HOST arrays of `count` DEVICE pointers (each as in btc_execute; C may be NULL when
 *                beta == 0).  Entries must not overlap one another's D.
 *   workspace    DEVICE memory, 256-byte aligned, btc_contraction_batched_workspace_size(count) bytes
 * Plans that run the tiled kernels serve the whole array with ONE launch (plus one split-K reduce):
 * the pointer array acts as a further batch dimension whose offsets are uploaded into the workspace
 * (a small host-to-device copy on the stream).  That path needs C[i] - C[0] == D[i] - D[0] for all i
 * (true for in-place updates and for C, D carved alike out of two pools) and returns NOT_SUPPORTED
 * otherwise.  Generic-kernel and Case 4 plans are executed entry by entry in stream order.
 * Nothing is allocated on the device.  The upload of the offsets is a copy from ordinary host memory,
 * which the CUDA runtime may start only after earlier work on the stream has finished (and which
 * cannot be part of a stream capture); apart from that the call does not wait for the device.
 * Errors: as btc_execute. */
btc_error_t btc_contraction_batched_workspace_size(btc_contraction_t op, int64_t count, size_t *bytes);
btc_error_t btc_execute_batched(btc_contraction_t op, void *cuda_stream, const void *alpha,
                                const void *const *A, const void *const *B, const void *beta,
                                const void *const *C, void *const *D, int64_t count,
                                void *workspace, size_t workspace_bytes);

/* Execute without allocating anything (the paper has no counterpart; this is a convenience of
 * this library).  Same operation and argument meaning as btc_execute with DEVICE pointers, but
 * the scratch that split-K plans need comes from an 8 MiB array that is part of the library's
 * device image instead of a caller workspace, and no status object is created: the call makes
 * no cudaMalloc / cudaFree, no host allocation and uses no allocating library routine.
 *
 * Who needs it: code that runs where device memory cannot be requested at that point -- a
 * plug-in inside a host application that handed all device memory to its own pool, a real-time
 * loop that may not pay for (or synchronise on) an allocation, a caller that only owns its
 * inputs and outputs -- and that has no workspace of its own to pass to btc_execute.
 *
 * Limits and rules:
 *   - operations whose btc_contraction_workspace_size exceeds 8 MiB (8 * 2^20 bytes) are refused
 *     with BTC_ERR_SCRATCH_LIMIT before anything is enqueued; use btc_execute for those;
 *   - the device that was current when the operation's handle was created must be current;
 *   - the first call on each device looks up the array's device address (set-up, once per
 *     device) and keeps it for the life of the process; make that first call before starting any
 *     stream capture, and do not reset the device (cudaDeviceReset) afterwards: the kept address
 *     would be stale;
 *   - after a bounded device-side wait gave up, the array may hold partial sums of an earlier call;
 *     the split-K reduction then leaves D untouched (poll BTC_ATTR_DEVICE_ERROR to find out);
 *   - all calls on one device share the one array, and it keeps whatever the last call left in
 *     it.  Nothing in it needs clearing (every partial sum is written before it is read), but
 *     two calls that may run on the GPU at the same time (different streams, different host
 *     threads) race on it: serialise them, e.g. by using one stream.
 * Errors: as btc_execute, plus SCRATCH_LIMIT. */
btc_error_t btc_execute_static_scratch(btc_contraction_t op, void *cuda_stream,
                                       const void *alpha, const void *A, const void *B,
                                       const void *beta, const void *C, void *D);

/* Status object (Sec. "Status Objects"): metadata of one execute call. */
enum {
    BTC_STATUS_KERNEL = 1,    /* int32: BTC_KERNEL_* that ran                 */
    BTC_STATUS_LAUNCHES = 2,  /* int32: kernels enqueued by the call          */
    BTC_STATUS_GRID = 3,      /* int32[3]                                      */
    BTC_STATUS_SPLIT_K = 4,   /* int32                                         */
    BTC_STATUS_VARIANT = 5    /* int32: tile variant of the tiled kernel that ran (-1: generic kernel); differs
                                 from BTC_ATTR_VARIANT when a bulk-copy variant met a base pointer that is
                                 not 16-byte aligned and its gathering twin ran instead */
};
btc_error_t btc_status_get(btc_status_t status, int32_t key, void *value, size_t len);
btc_error_t btc_destroy_status(btc_status_t *status);

/* ---- Binary and unary operations (Sec. "Unary and Binary Operations") --------------------------
 *
 *     C := alpha * op(A) + beta * op(B)
 *
 * B and C carry the same labels (labelsC; B has C's rank and extents, its strides are its own).
 * A label in A and C is matched; a label only in A is summed over (reduction); along a label only
 * in C the value of A is repeated (broadcast); a label repeated inside A addresses its
 * (semi-)diagonal elements (one mode whose stride is the sum of the occurrences' strides, Note 6).
 * Unary scaling / permutation B := alpha A is the case beta = 0 (pass B = NULL).  op conjugates
 * complex operands when the flag is set.  All tensors share one element type.
 *
 * btc_create_elementwise validates (extents per label, B against C, no repeated label and no
 * aliasing inside C) and plans once; btc_elementwise_execute takes device pointers (each the
 * address of logical element (0,...,0)), host scalars (NULL = the values given at creation) and a
 * CUDA stream, allocates nothing and does not synchronise.  beta == 0: B is not read; alpha == 0:
 * A is not read.  B may be the same memory as C only with identical strides (in place).
 * Errors: BTC_ERR_EXTENT_MISMATCH, BTC_ERR_C_D_MISMATCH (B does not match C), BTC_ERR_D_ALIASING
 * (elements of C alias), BTC_ERR_NOT_SUPPORTED (label repeated in C, mixed types),
 * BTC_ERR_MISALIGNED, BTC_ERR_CUDA. */
typedef struct btc_elementwise_s *btc_elementwise_t;
btc_error_t btc_create_elementwise(btc_handle_t handle,
                                   btc_tensor_info_t A, const int64_t *labelsA, int conjA,
                                   btc_tensor_info_t B, int conjB,
                                   btc_tensor_info_t C, const int64_t *labelsC,
                                   const void *alpha, const void *beta, btc_elementwise_t *out);
btc_error_t btc_destroy_elementwise(btc_elementwise_t *op);
btc_error_t btc_elementwise_execute(btc_elementwise_t op, void *cuda_stream, const void *alpha, const void *A,
                                    const void *beta, const void *B, void *C);
enum {
    BTC_EW_ATTR_KERNEL = 1,    /* int32, read: the planned kernel.  1 = one thread (or warp) per element
                                  of C, 2 = tiles through shared memory (input and output contiguous
                                  along different labels; 128 x 64 elements of 4 bytes, 64 x 64 of 8,
                                  32 x 32 of 16)                                                 */
    BTC_EW_ATTR_NUM_MODES = 2, /* int32[2], read: loop dimensions over C and summed dimensions after
                                  merging                                                        */
    BTC_EW_ATTR_LAST_KERNEL = 3 /* int32, read: the kernel the last execute launched (0 before the
                                  first): 1, 2 as above, 3 = 16-byte vectors along C's contiguous
                                  label, chosen at execute time when strides and pointers allow  */
};
btc_error_t btc_elementwise_get_attr(btc_elementwise_t op, int32_t key, void *value, size_t len, size_t *needed);

/* Peak micro-benchmarks (no counterpart in the paper; the paper leaves benchmarks to future work, Sec.
 * "Outlook").  Measures what this device sustains with a kernel that does nothing else, so that the
 * roofline fraction of a contraction can be quoted against a figure taken on the same device in the
 * same run.  Arithmetic kinds run register-resident loops of independent FMA / MMA chains and need no
 * buffer (`buffer` may be NULL); memory kinds make one pass of 16-byte accesses over the caller's
 * DEVICE buffer of `bytes` bytes (16-byte aligned, at least 1 MiB; the copy reads the first half and
 * writes the second; use more than the L2 size for a DRAM figure).  One untimed launch, then `repeats`
 * timed launches between two CUDA events on `cuda_stream`; the call waits for them.  *value = flop/s
 * (two per FMA) or byte/s (copy: bytes read + bytes written).  Allocates nothing on the device.
 * Errors: INVALID_ARGUMENT, CUDA. */
enum {
    BTC_PEAK_FP64_FMA = 0,      /* DFMA, 16 independent chains per thread                         */
    BTC_PEAK_FP32_FMA = 1,      /* FFMA likewise                                                  */
    BTC_PEAK_FP64_MMA_K16 = 2,  /* mma.sync m16n8k16 f64: the FP64 tensor pipe the fp64 kernels use */
    BTC_PEAK_FP64_MMA_K4 = 3,   /* mma.sync m8n8k4 f64                                            */
    BTC_PEAK_TF32_MMA_SYNC = 4, /* mma.sync m16n8k8 tf32: the warp-level tensor path              */
    BTC_PEAK_HBM_READ = 5,
    BTC_PEAK_HBM_WRITE = 6,
    BTC_PEAK_HBM_COPY = 7
};
btc_error_t btc_measure_peak(btc_handle_t handle, int32_t which, void *cuda_stream, void *buffer, size_t bytes,
                             int32_t repeats, double *value);

/* Self-test of the device-side failure detection (no counterpart in the paper).  Every wait inside
 * the kernels is bounded: after a fixed number of polls it gives up, records a code in the
 * operation's device error word (BTC_ATTR_DEVICE_ERROR) and lets the kernel return.  This call
 * launches one small kernel on `cuda_stream` whose 64 threads wait, with a limit of `polls`
 * (1..65536) polls, on a barrier that nothing ever signals, waits for it, and reports through
 * *error_code the code the wait recorded (non-zero) and through *threads_gave_up how many
 * threads gave up (64).  Nothing faults or traps; the CUDA context stays usable.  Allocates and
 * frees 8 bytes of device memory. */
btc_error_t btc_selftest_bounded_wait(btc_handle_t handle, void *cuda_stream, int32_t polls,
                                      int32_t *error_code, int32_t *threads_gave_up);

/* Text for an error code (the strerror analogue of Sec. "Error Handling").  Writes at most `len`
 * bytes including the terminator; *needed (if not NULL) receives the full length. */
btc_error_t btc_explain_error(btc_error_t code, char *buf, size_t len, size_t *needed);

#ifdef __cplusplus
}
#endif
#endif /* BTC_H_ */
