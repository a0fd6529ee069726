// Host-side planner of the contraction library: validation, label classification, repeated-label
// merge, mode fusion, operand role choice, loop ordering and offset tables.
//
// Follows Sec. "Operations" (label classes H, F_A, F_B, P; Cases 1-4), Note 6 (repeated labels
// add their strides) and the checks listed in Sec. "Algorithm Structure".  Everything here is
// integer work that runs once per operation object.
#pragma once

#include <cstdint>
#include <string>
#include <vector>

#include "../../include/btc.h"

namespace btc {

struct TensorDesc {
    btc_dtype_t dtype = BTC_F64;
    std::vector<int64_t> extent, stride;
};

// One loop dimension after merging/fusing: its extent and its element stride in each tensor
// (0 where the tensor does not carry it).  After a role swap "A" means the operand that plays
// the M side.
struct Mode {
    int64_t extent = 1;
    int64_t sA = 0, sB = 0, sD = 0;
};

enum class LoadDir : int32_t { ALONG_FREE = 0, ALONG_K = 1 };

struct TileConfig {
    int32_t bm = 0, bn = 0, bk = 0;   // CTA tile in elements of the operation's dtype
    int32_t threads = 0;
    int32_t stages = 0;
    int32_t variant = 0;              // index into the kernel table
};

struct Plan {
    btc_dtype_t dtype = BTC_F64;
    bool conjA = false, conjB = false, conjC = false;  // in planned roles (after swap)
    bool swapped = false;        // true: the caller's B is the plan's A
    bool has_c_desc = false;
    bool has_isolated = false;   // Case 4 labels present; if planned as they are, the generic kernel sums them
    // element types differ between the tensors (same part width; D complex when an input is): which of the
    // planned A, B and C are complex.  Such operations run on the per-element kernel.
    bool mixed = false, cplxA = false, cplxB = false, cplxC = false;

    // loop dimensions in planned order, first entry fastest in the linearised index
    std::vector<Mode> batch, m, n, k;
    int64_t Bt = 1, M = 1, N = 1, K = 1;

    // tile-kernel decisions
    int32_t kernel = BTC_KERNEL_GENERIC;
    TileConfig tile;
    int32_t split_k = 1;
    LoadDir dirA = LoadDir::ALONG_FREE, dirB = LoadDir::ALONG_FREE;
    int32_t vecA = 1, vecB = 1;          // elements per global load that the strides allow
    int32_t vecD = 1;                    // 4: groups of four consecutive m are 16 aligned bytes of D
    int64_t alignA = 1, alignB = 1;      // required base-pointer alignment (bytes) for vecA / vecB
    // any element type: groups of 16 bytes along the first M mode are contiguous, 16-byte aligned (given an aligned
    // base) and whole in D / in A (what the streaming kernel for K <= 4 needs for its vector accesses)
    bool rows16D = false, rows16A = false;

    // element-offset tables (host copies; the API object uploads them)
    std::vector<int64_t> offA_m, offD_m, offB_n, offD_n, offA_k, offB_k, offA_h, offB_h, offD_h;

    // memory span of each caller-side tensor in elements relative to its base pointer
    int64_t spanA_lo = 0, spanA_hi = 0, spanB_lo = 0, spanB_hi = 0, spanD_lo = 0, spanD_hi = 0;

    std::string describe() const;
};

struct PlanRequest {
    TensorDesc A, B, C, D;
    bool has_c = false;
    std::vector<int64_t> labelsA, labelsB, labelsC, labelsD;
    bool conjA = false, conjB = false, conjC = false;
    int32_t force_kernel = BTC_KERNEL_AUTO;
    int32_t force_split_k = 0;   // 0 = choose
    int32_t force_variant = -1;  // -1 = choose; otherwise index of the tile variant for the dtype
    int32_t strict_fp32 = 0;     // 1: fp32 / complex64 products and sums in IEEE fp32 (no TF32 split); 2: sums kept in fp64
    int32_t batch_hint = 1;      // pointer-array entries the operation is expected to run with at a time
    int32_t sm_count = 148;
};

// Validates the request and fills `plan`.  Returns a btc_error_t.
int make_plan(const PlanRequest &req, Plan &plan);

// The M-side operand seen as a tensor of at most five dimensions in which every (tile of `bm`
// rows) x (stage of `bk` contracted indices) is one rectangular box, so that a single bulk tensor
// copy (cp.async.bulk.tensor) can fetch it.  Exists when the tile's rows are whole leading M modes
// (at most one of them partly), a stage is a whole number of entries of the first contracted
// mode, the operand is contiguous along the first M mode or the first contracted mode, and all
// other strides are positive multiples of 16 bytes.  Loop dimensions whose strides chain in this
// operand share one dimension, which is how the tile index, the stage index and the batch index
// usually collapse into a few coordinates.
struct TmaOperand {
    bool ok = false;
    bool k_major = false;                 // dimension 0 is the contracted index (else the first M mode)
    uint64_t dim[5] = {1, 1, 1, 1, 1};    // extents in elements, dimension 0 contiguous
    uint64_t stride[5] = {1, 0, 0, 0, 0}; // element strides
    uint32_t box[5] = {1, 1, 1, 1, 1};
    int32_t rank = 0;                     // dimensions in use (the rest have extent 1)
    // box origin = coordM[tile of M] + coordK[stage] + coordH[batch entry], five entries each
    std::vector<int32_t> coordM, coordK, coordH;
};
bool make_tma_operand(const Plan &plan, int bm, int bk, TmaOperand &out);

// Case 4: the sum over the labels that occur in one input only, taken before the contraction.
struct IsolatedSum {
    bool active = false;
    // loop dimensions of the input tensor (repeated labels merged), smallest |stride| first
    std::vector<int64_t> keep_ext, keep_str, iso_ext, iso_str;
    int64_t total_keep = 1, total_iso = 1;
    bool lanes_over_iso = false;   // the isolated index is the more contiguous one: one warp per result element
};

// For a validated request: `inner` = the same contraction on A' and B', the inputs summed over
// their isolated labels (dense, kept labels in order of increasing |stride| in the input; an
// input without isolated labels is passed through), and how to form A' and B'.
void split_isolated(const PlanRequest &req, PlanRequest &inner, IsolatedSum &sumA, IsolatedSum &sumB);

// ---- binary / unary operation  C := alpha op(A) + beta op(B)  (Sec. "Unary and Binary Operations")
struct ElementwiseRequest {
    TensorDesc A, B, C;
    bool has_b = false;
    std::vector<int64_t> labelsA, labelsC;   // B carries C's labels
    bool conjA = false, conjB = false;
};

enum class ElementwiseKernel : int32_t { DIRECT = 1, TRANSPOSING = 2 };

struct ElementwisePlan {
    btc_dtype_t dtype = BTC_F64;
    bool conjA = false, conjB = false, has_b = false;
    // loop dimensions over C (labels of C; sA = 0 where A is broadcast), smallest |stride in C|
    // first, and the summed dimensions (labels only in A; only sA is used), smallest |sA| first
    std::vector<Mode> keep, sum;
    int64_t total_keep = 1, total_sum = 1;
    ElementwiseKernel kernel = ElementwiseKernel::DIRECT;
    int32_t tile_mode_a = 0;      // TRANSPOSING: index in `keep` of the dimension along which A is read
                                  // (C is written along dimension 0)
    int64_t spanA_lo = 0, spanA_hi = 0, spanB_lo = 0, spanB_hi = 0, spanC_lo = 0, spanC_hi = 0;
};

// Validates the request and fills `plan`.  Returns a btc_error_t.
int make_elementwise_plan(const ElementwiseRequest &req, ElementwisePlan &plan);

size_t dtype_size(btc_dtype_t t);
bool dtype_is_complex(btc_dtype_t t);

// Largest total number of table entries the tiled kernels accept before the planner falls back
// to the generic kernel.
constexpr int64_t kMaxTableEntries = int64_t(1) << 26;

}  // namespace btc
