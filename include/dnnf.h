/*
 * dnnf.h -- C ABI of the fused operator-block executor.
 *
 * The library takes a computational graph (operators with type and parameters,
 * tensors, data-flow; paper Section 4.1), annotates every operator with its
 * mapping type (Section 3.1, Table 2) to form the Extended Computational Graph,
 * optionally rewrites it with mathematical-property rules (Section 4.2,
 * Table 4), groups operators into fusion blocks (Section 4.3, Listing 1,
 * Table 3) and runs every block as ONE CUDA kernel that keeps the block's
 * intermediates in registers / shared memory / tensor memory (Section 4.4).
 *
 * Conventions
 *  - Every function returns a dnnf_status_t; DNNF_OK is 0.  No exception crosses
 *    this boundary; a failed call leaves the graph usable and stores a message
 *    retrievable with dnnf_last_error().
 *  - Pointers named host_* are host memory; pointers named dev_* are device
 *    memory owned by the caller.  The library never allocates device memory and
 *    never synchronises inside dnnf_run().
 *  - Tensors are dense, row-major (last dimension contiguous).
 *  - Call order: create -> add_tensor/add_op/mark_output -> [rewrite] -> plan ->
 *    bind/bind_workspace -> run.  add_* after plan returns DNNF_ERR_STATE.
 *  - A handle is not thread-safe; distinct handles are independent.
 *  - There is no CPU fallback: a block with no kernel family makes dnnf_plan()
 *    fail with DNNF_ERR_UNSUPPORTED_OP.
 */
#ifndef DNNF_H_
#define DNNF_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define DNNF_API __attribute__((visibility("default")))
#else
#define DNNF_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dnnf_graph dnnf_graph;   /* opaque; freed by dnnf_graph_destroy */

typedef enum {
  DNNF_OK = 0,
  DNNF_ERR_INVALID_ARG = 1,
  DNNF_ERR_SHAPE = 2,
  DNNF_ERR_UNSUPPORTED_OP = 3,
  DNNF_ERR_STATE = 4,
  DNNF_ERR_UNBOUND = 5,
  DNNF_ERR_WORKSPACE = 6,
  DNNF_ERR_CUDA = 7,
  DNNF_ERR_TIMEOUT = 8
} dnnf_status_t;

typedef enum { DNNF_F32 = 0, DNNF_BF16 = 1 } dnnf_dtype_t;
typedef enum { DNNF_INPUT = 0, DNNF_WEIGHT = 1 } dnnf_tensor_kind_t;

/* The five mapping types of Section 3.1, in the paper's order of increasing
 * complexity (used to type an operator with mixed input/output pairs). */
typedef enum {
  DNNF_ONE_TO_ONE = 0, DNNF_REORGANIZE = 1, DNNF_SHUFFLE = 2,
  DNNF_ONE_TO_MANY = 3, DNNF_MANY_TO_MANY = 4
} dnnf_mapping_t;

/* Table 3 cell colours. */
typedef enum { DNNF_FUSE_THROUGH = 0 /*green*/, DNNF_FUSE_DEPEND = 1 /*yellow*/, DNNF_FUSE_BREAK = 2 /*red*/ } dnnf_fuse_t;

/* Operator vocabulary (ONNX names as classified in Table 2, plus the
 * element-wise operators Table 4 uses). */
typedef enum {
  DNNF_OP_ADD = 1, DNNF_OP_SUB, DNNF_OP_MUL, DNNF_OP_DIV,
  DNNF_OP_MULC, DNNF_OP_ADDC,                       /* scalar attribute C */
  DNNF_OP_SIGMOID, DNNF_OP_TANH, DNNF_OP_ERF, DNNF_OP_EXP, DNNF_OP_LOG, DNNF_OP_SQRT,
  DNNF_OP_ABS, DNNF_OP_NEG, DNNF_OP_RECIP, DNNF_OP_SQUARE, DNNF_OP_RELU,
  DNNF_OP_CLIP,                                     /* attributes LO, HI */
  DNNF_OP_POW,                                      /* attribute P */
  DNNF_OP_GELU,                                     /* attribute APPROX: 0 erf, 1 tanh */
  DNNF_OP_SCALESHIFT,                               /* (x, scale[c], shift[c]); attribute AXIS */
  DNNF_OP_TRANSPOSE,                                /* attribute PERM */
  DNNF_OP_RESHAPE,                                  /* attribute SHAPE (one -1 allowed) */
  DNNF_OP_FLATTEN, DNNF_OP_SQUEEZE, DNNF_OP_UNSQUEEZE, /* attribute AXIS / AXES */
  DNNF_OP_SPLIT,                                    /* attributes AXIS, SIZES; several outputs */
  DNNF_OP_SLICE,                                    /* attributes AXIS, START, END */
  DNNF_OP_MATMUL,
  DNNF_OP_CONV1X1,                                  /* NHWC x [Cin,Cout] */
  DNNF_OP_DWCONV3X3,                                /* NHWC x [3,3,C], stride 1, zero pad 1 */
  DNNF_OP_SOFTMAX,                                  /* attribute AXIS (last axis only) */
  DNNF_OP_LAYERNORM,                                /* (x, gamma, beta), or (x) alone for no scale and shift; attributes AXIS, EPS */
  DNNF_OP_REDUCESUM, DNNF_OP_REDUCEMEAN, DNNF_OP_REDUCEMAX, DNNF_OP_REDUCEPROD, /* AXIS (last), KEEPDIMS */
  DNNF_OP_EXPAND,                                   /* attribute SHAPE */
  DNNF_OP_BITSHIFT,                                 /* attribute BITS; planning/rewriting only */
  /* Table 2 operators that are index maps of an NHWC tensor [N,H,W,C].  dnnf_add_op records them in the ECG as the
   * Reshape / Transpose / Expand operators they are made of, the way a Split becomes Slices, so that they fuse
   * into their neighbours as changed load and store indices (Section 4.4.2):                                     */
  DNNF_OP_DEPTHTOSPACE,                             /* Shuffle; attribute BLOCK b: y[n,h*b+i,w*b+j,c] = x[n,h,w,(i*b+j)*C/b^2+c] */
  DNNF_OP_SPACETODEPTH,                             /* Shuffle; attribute BLOCK b: the inverse map */
  DNNF_OP_RESIZE,                                   /* One-to-Many; nearest neighbour, integer attribute SCALE s:
                                                       y[n,h,w,c] = x[n,h/s,w/s,c] */
  DNNF_OP_CONCAT,                                   /* One-to-One (Table 2); 2 to 4 inputs, attribute AXIS.  Recorded as one
                                                       ConcatPart per input: each writes its input's values into its
                                                       range of the result, which all parts share in place, so that an
                                                       input's producer block stores straight into the result (the
                                                       Concat becomes changed store indices, Section 4.4.2) */
  DNNF_OP_MAXPOOL, DNNF_OP_AVGPOOL,                 /* Many-to-Many (Table 2); NHWC fp32; attributes KERNEL k, STRIDE s, PAD p < k:
                                                       result [N,(H+2p-k)/s+1,(W+2p-k)/s+1,C]; MaxPool ignores the padding,
                                                       AveragePool divides by the number of elements inside the image;
                                                       a global pool is KERNEL = H = W, STRIDE 1, PAD 0 */
  /* more One-to-One operators of Table 2 */
  DNNF_OP_SIN, DNNF_OP_COS, DNNF_OP_ASIN, DNNF_OP_CEIL, DNNF_OP_FLOOR,
  DNNF_OP_ROUND,                                    /* to nearest, ties to even */
  DNNF_OP_LEAKYRELU,                                /* attribute C: the slope for negative inputs */
  DNNF_OP_NOT,                                      /* on 0 / 1 valued tensors: 1 where the input is 0, else 0 */
  DNNF_OP_GREATER,                                  /* (a, b) with broadcasting: 1 where a > b, else 0 */
  DNNF_OP_PRELU,                                    /* (x, slope) with broadcasting: x where x > 0, else slope * x */
  DNNF_OP_CONVTRANSPOSE,                            /* Many-to-Many; NHWC x [Cin,k,k,Cout], attributes KERNEL k, STRIDE s <= k (default: k) and PAD
                                                       p < k: y[n,h*s+i-p,w*s+j-p,o] += sum_c x[n,h,w,c] W[c,i,j,o], the result has
                                                       (H-1)*s + k - 2p rows.  With s = k and p = 0 the patches do not overlap and the operator is
                                                       recorded as Reshape(W) -> Conv1x1 -> DepthToSpace; otherwise as Reshape(W) -> Conv1x1
                                                       (all k*k*Cout patch values of every pixel) -> Col2Im (each output element adds the at most
                                                       ceil(k/s)^2 patch values that land on it; Cout a multiple of 4) */
  DNNF_OP_GATHER,                                   /* One-to-Many; (table [V,D], indices [...]) along axis 0: y[..., :] = table[indices[...], :].
                                                       Indices are integer-valued fp32 numbers; out-of-range ones are clamped.  A table of
                                                       another rank or another AXIS is recorded as Transpose / Reshape to that form, the
                                                       row gather, and Reshape / Transpose of the result (the index axes take the place of
                                                       the gathered axis) */
  DNNF_OP_WHERE,                                    /* One-to-One (Table 2); (cond, a, b) with broadcasting: a where the 0 / 1 valued cond
                                                       is non-zero, else b.  A selection: the other branch's value is never touched */
  DNNF_OP_CAST,                                     /* One-to-One (Table 2); attribute TO: DNNF_CAST_F32 (values unchanged), DNNF_CAST_BF16
                                                       (nearest bfloat16, ties to even; the result tensor is bf16), DNNF_CAST_I32 (the integer
                                                       toward zero) or DNNF_CAST_BOOL (1 where non-zero, else 0); integer and boolean
                                                       results are stored as fp32 numbers with those values */
  DNNF_OP_CUMSUM,                                   /* Many-to-Many (Table 2); running sum along the last axis (attribute AXIS must name it);
                                                       attributes EXCLUSIVE (sum of the elements before) and REVERSE (from the far end) */
  DNNF_OP_INSTANCENORM,                             /* Many-to-Many (Table 2); (x NHWC, scale[C], shift[C]), attribute EPS: each image and
                                                       channel is normalised by the mean and biased variance over its H x W positions,
                                                       then scaled and shifted per channel; C a multiple of 4 */
  DNNF_OP_EINSUM,                                   /* Many-to-Many (Table 2); two operands, attributes LABELS_A, LABELS_B, LABELS_OUT: one small
                                                       integer per axis (the letters of "bhqd,bhkd->bhqk").  Every label of the result comes
                                                       from an operand, a label of both operands that is missing in the result is summed
                                                       over (at least one), no label repeats inside an operand and none belongs to one
                                                       operand only without reaching the result.  Recorded as Transpose / Reshape of the
                                                       operands -> (batched) MatMul -> Reshape / Transpose, which it equals term by term */
  DNNF_OP_COL2IM,                                   /* internal (made by ConvTranspose): ([N,H,W,k*k*C]); KERNEL, STRIDE, PAD; Many-to-Many */
  DNNF_OP_CONCATPART,                               /* internal (made by Concat): (x [, result so far]); AXIS, START, SHAPE */
  DNNF_OP__COUNT
} dnnf_op_t;

typedef enum {
  DNNF_ATTR_C = 1, DNNF_ATTR_LO, DNNF_ATTR_HI, DNNF_ATTR_P, DNNF_ATTR_EPS,   /* use f */
  DNNF_ATTR_APPROX, DNNF_ATTR_AXIS, DNNF_ATTR_KEEPDIMS, DNNF_ATTR_START, DNNF_ATTR_END, DNNF_ATTR_BITS, /* use i[0] */
  DNNF_ATTR_PERM, DNNF_ATTR_SHAPE, DNNF_ATTR_SIZES, DNNF_ATTR_AXES,           /* use i[0..n) */
  DNNF_ATTR_BLOCK, DNNF_ATTR_SCALE, DNNF_ATTR_KERNEL, DNNF_ATTR_STRIDE, DNNF_ATTR_PAD,  /* use i[0] */
  DNNF_ATTR_TO, DNNF_ATTR_EXCLUSIVE, DNNF_ATTR_REVERSE,                                   /* use i[0] */
  DNNF_ATTR_LABELS_A, DNNF_ATTR_LABELS_B, DNNF_ATTR_LABELS_OUT                            /* use i[0..n) */
} dnnf_attr_key_t;

/* Cast targets (attribute TO) */
#define DNNF_CAST_F32   0
#define DNNF_CAST_BF16  1
#define DNNF_CAST_I32   2
#define DNNF_CAST_BOOL  3

typedef struct {
  int32_t key;      /* dnnf_attr_key_t */
  int32_t n;        /* number of valid entries in i[] */
  int64_t i[8];
  double  f;
} dnnf_attr;

/* dnnf_rewrite flags */
#define DNNF_REWRITE_DEFAULT        0u
#define DNNF_REWRITE_NONE           1u   /* leave the graph as given */
#define DNNF_REWRITE_CANON_MACRO    2u   /* also fold the 9-operator LayerNorm expansion into one LayerNorm
                                            operator (an extension beyond the paper's printed rules) */
#define DNNF_REWRITE_KEEP_LAYOUT    4u   /* skip the layout selection of Section 4.4.2: leave every Transpose where the graph
                                            has it (by default element-wise operators and batch normalisation take the layout
                                            of the convolution, pool, GEMM or Softmax they feed, and Transposes that then
                                            meet their inverse disappear) */
/* dnnf_plan flags */
#define DNNF_PLAN_FUSED             0u
#define DNNF_PLAN_UNFUSED           1u   /* one block per operator: the no-fusion baseline of Section 5 ("OurB") */
#define DNNF_PLAN_STRICT_TABLE3     2u   /* type a broadcast operand's consumer One-to-Many on every edge */
#define DNNF_PLAN_ALLOW_PROLOGUE    4u   /* planning only: let One-to-One predecessors fuse in front of a
                                            GEMM/conv anchor (Listing 1 literal); such plans cannot be run */
#define DNNF_PLAN_BEYOND_TABLE3      8u   /* an extension beyond the paper's rules: MatMul -> [scale] -> [+ mask] -> Softmax ->
                                            MatMul runs as ONE kernel, and so does Conv1x1 -> DwConv3x3 -> Conv1x1 with
                                            their chains (Table 3 marks Many-to-Many followed by Many-to-Many red, so the
                                            default plan keeps three blocks each) */
/* Kernel-selection overrides.  The plan, its blocks and the results stay the same; a block is only lowered to another
 * kernel of its family.  They exist so that every kernel, including the ones the planner rarely picks, can be
 * tested and timed through this interface; the library reads no environment variable. */
#define DNNF_PLAN_SPLIT_ALWAYS      0x100u   /* cut fp32 contractions into K slices / column blocks wherever that is possible,
                                                not only where the cost model says it pays */
#define DNNF_PLAN_NO_K_SLICES       0x200u   /* never cut an fp32 contraction along K */
#define DNNF_PLAN_NO_COLUMN_BLOCKS  0x400u   /* never cut an fp32 contraction into column blocks */
#define DNNF_PLAN_NO_TF32_GEMM      0x800u   /* fp32 contractions on the FMA pipes instead of split-TF32 tensor-core kernels */
#define DNNF_PLAN_NO_PAIR_GEMM      0x1000u  /* bf16 GEMM blocks without the CTA-pair kernel */
#define DNNF_PLAN_NO_SPLIT_K        0x2000u  /* bf16 GEMM blocks without a split over K */
#define DNNF_PLAN_NO_TMA_DWCONV     0x4000u  /* depthwise convolutions without the TMA-tiled kernel */
#define DNNF_PLAN_NO_TILE_GEMM      0x8000u  /* bf16 GEMM blocks without the one-tile-per-CTA kernel */
#define DNNF_PLAN_NO_SMALL_CONV     0x40000u /* fp32 contractions with few rows without the one-tile-per-CTA mma.sync kernel */
#define DNNF_PLAN_MBCONV_ALWAYS     0x20000u /* with DNNF_PLAN_BEYOND_TABLE3: form the single-kernel inverted-residual block whatever its
                                                size (by default only while its 8 x 16 pixel tiles fit one wave of CTAs, where it was
                                                measured faster than the three kernels; this flag changes the plan, not only a kernel) */
#define DNNF_PLAN_CLUSTER_SPLIT_K   0x10000u /* one-tile-per-CTA kernel: clusters of 2 or 4 CTAs share a tile's k-tiles and add their
                                                partial sums through distributed shared memory (measured slower at the sizes
                                                tried, so not the default) */

typedef struct {
  int32_t ops_before, ops_after;
  int64_t flops_before, flops_after;       /* Table 4's #FLOPS model */
  int32_t rules_applied;
  int32_t applied_by_rule[16];             /* index: see dnnf_rule_name() */
  int32_t folded_constants;
  int32_t layout_transposes_removed;       /* Transposes the layout selection took out of the graph */
} dnnf_rewrite_stats;

typedef struct {
  int32_t n_ops;               /* original operators (a Split counts once) */
  int32_t n_blocks;            /* fusion blocks */
  int32_t n_kernels;           /* blocks that launch a kernel (an isolated Reshape launches none) */
  double  fusion_rate;         /* n_ops / n_blocks (Section 5.2) */
  int64_t irs_bytes_unfused;   /* bytes of all operator outputs that are not graph outputs */
  int64_t irs_bytes_fused;     /* bytes of intermediates still materialised between blocks */
  int64_t workspace_bytes;
  int32_t n_yellow_decisions;  /* Table 3 yellow cells resolved by the cost model */
  int32_t n_yellow_fused;
  int32_t n_profile_hits;      /* candidate-block costs answered by the profiling database */
  int32_t n_profile_misses;    /* distinct candidate signatures it did not have (analytic cost used) */
} dnnf_plan_stats;

typedef enum {
  DNNF_FAMILY_ALIAS = 0,       /* pure Reorganize: zero-copy */
  DNNF_FAMILY_ELEMENTWISE = 1, /* One-to-One / broadcast chain, contiguous */
  DNNF_FAMILY_TRANSPOSE = 2,   /* chain with a Shuffle staged through shared memory */
  DNNF_FAMILY_ROW = 3,         /* chain around a last-axis reduction (Softmax, LayerNorm, Reduce*) */
  DNNF_FAMILY_GEMM = 4,        /* tensor-core GEMM anchor with an epilogue chain */
  DNNF_FAMILY_CONV1X1 = 5,     /* fp32 pointwise convolution with an epilogue chain */
  DNNF_FAMILY_DWCONV = 6,      /* fp32 depthwise 3x3 with an epilogue chain */
  DNNF_FAMILY_POOL = 7,        /* fp32 MaxPool / AveragePool with an epilogue chain */
  DNNF_FAMILY_GATHER = 8,      /* row gather by an index tensor */
  DNNF_FAMILY_ATTENTION = 9,   /* scores, softmax and weighted sum of a head in one kernel (DNNF_PLAN_BEYOND_TABLE3 only) */
  DNNF_FAMILY_INSTNORM = 11,   /* fp32 InstanceNormalization with an epilogue chain */
  DNNF_FAMILY_MBCONV = 10      /* pointwise expansion, depthwise 3x3 and pointwise projection of an inverted-residual block in one
                                  kernel, the expanded tensor kept in shared memory (DNNF_PLAN_BEYOND_TABLE3 only) */
} dnnf_family_t;

typedef struct {
  int32_t family;              /* dnnf_family_t */
  int32_t mapping;             /* dnnf_mapping_t of the fused block */
  int32_t n_ops;
  int32_t op_kinds[48];        /* dnnf_op_t of the first 48 operators */
  int32_t n_inputs, n_outputs;
  int64_t bytes_in, bytes_out; /* algorithmic HBM bytes: each external input/output once */
  int64_t flops;               /* 2*M*N*K for contraction anchors, else 0 */
  int32_t n_microops;
  int32_t grid, threads;
  int32_t variant;             /* kernel specialisation chosen (family-specific) */
} dnnf_block_desc;

/* ---- graph construction (Section 4.1: the computational graph handed over by a
 *      host framework) ------------------------------------------------------- */

/* Creates an empty graph.  *out is owned by the library until dnnf_graph_destroy. */
DNNF_API int dnnf_graph_create(dnnf_graph** out);
DNNF_API int dnnf_graph_destroy(dnnf_graph* g);

/* Declares an external tensor (model input or weight).  host_dims has `rank`
 * entries (rank <= 6).  Returns its id in *tensor_id. */
DNNF_API int dnnf_add_tensor(dnnf_graph* g, const char* name, int dtype, int rank,
                    const int64_t* host_dims, int kind, int* tensor_id);

/* Appends an operator.  host_in_ids are ids returned earlier; outputs are created
 * by shape inference and their ids written to host_out_ids (capacity max_out),
 * their count to *n_out.  The operator is tagged with its mapping type
 * (Table 2; an operator with mixed input/output pairs takes the most complex
 * one, Section 3.1).  Output dtype is the dtype of input 0. */
DNNF_API int dnnf_add_op(dnnf_graph* g, int op_kind, int n_in, const int* host_in_ids,
                const dnnf_attr* host_attrs, int n_attrs,
                int max_out, int* host_out_ids, int* n_out);

/* Marks a tensor as a result the caller wants (never removable, Section 3.2
 * "IR_removable"). */
DNNF_API int dnnf_mark_output(dnnf_graph* g, int tensor_id);

/* Tensor introspection: rank and dims (capacity 6), dtype. */
DNNF_API int dnnf_tensor_info(const dnnf_graph* g, int tensor_id, int* dtype, int* rank, int64_t* host_dims);
/* Mapping type the ECG holds for operator `op_index` (insertion order). */
DNNF_API int dnnf_op_mapping(const dnnf_graph* g, int op_index, int* mapping);

/* ---- Table 3 ------------------------------------------------------------------ */

/* Mapping-type analysis of fusing `first` then `second` (both dnnf_mapping_t):
 * writes the fused block's mapping type and the cell colour. */
DNNF_API int dnnf_mapping_check(int first, int second, int* fused_mapping, int* colour);

/* ---- Section 4.2: mathematical-property graph rewriting ------------------------ */

/* Partitions the graph at operators with no associative/commutative/distributive
 * property, matches the printed rules of Table 4 inside each partition, applies
 * the match with the largest #FLOPS reduction and repeats to a fixed point.
 * stats may be NULL. */
DNNF_API int dnnf_rewrite(dnnf_graph* g, uint32_t flags, dnnf_rewrite_stats* host_stats);
DNNF_API const char* dnnf_rule_name(int rule_index);

/* ---- Section 4.3: fusion-plan generation ---------------------------------------- */

/* Listing 1: seed = One-to-One operator with the smallest intermediate result;
 * grow along successors, then predecessors, consulting Table 3 (green: fuse,
 * red: stop, yellow: cost model) and a constraint check; repeat over seeds.
 * Then lowers every block to one kernel launch (data-flow-tree traversal of
 * Section 4.4).  stats may be NULL. */
DNNF_API int dnnf_plan(dnnf_graph* g, uint32_t flags, dnnf_plan_stats* host_stats);
DNNF_API int dnnf_block_count(const dnnf_graph* g, int* n_blocks);
DNNF_API int dnnf_block_info(const dnnf_graph* g, int block, dnnf_block_desc* host_out);
/* External tensors of a planned block: what it reads from and writes to memory (ids as returned by dnnf_add_tensor /
 * dnnf_add_op; capacities in entries, counts always written). */
DNNF_API int dnnf_block_tensors(const dnnf_graph* g, int block, int* host_in_ids, int cap_in, int* n_in,
                                int* host_out_ids, int cap_out, int* n_out);
/* Where a tensor lives after dnnf_plan: *where = 0 caller-bound (external input or marked output), 1 in the workspace at
 * *workspace_offset bytes, 2 nowhere (it stays inside its block: IR_removable, Section 3.2), 3 it shares the caller-bound
 * storage of tensor *workspace_offset (a zero-copy Reshape).  With dnnf_run_block this lets a caller feed one block with
 * inputs of its own and read its results (per-block parity tests, per-block timing on chosen data). */
DNNF_API int dnnf_tensor_location(const dnnf_graph* g, int tensor_id, int* where, int64_t* workspace_offset);
/* Writes the block's micro-op program as text ("MOV in0; ADD in1; MUL c0=0.5; ...")
 * into host_buf (capacity bytes, NUL-terminated, truncated if needed): the linearised
 * data-flow tree of Section 4.4, every value computed once. */
DNNF_API int dnnf_block_program(const dnnf_graph* g, int block, char* host_buf, size_t capacity);
/* Block index that holds operator `op_index` (insertion order), after dnnf_plan. */
DNNF_API int dnnf_op_block(const dnnf_graph* g, int op_index, int* block);
/* Number of operators currently alive (after rewriting) and their kinds. */
DNNF_API int dnnf_op_count(const dnnf_graph* g, int* n_ops);
DNNF_API int dnnf_op_kind(const dnnf_graph* g, int op_index, int* kind, int* alive);

/* ---- profiling database (Section 4.3: "fusion profitability ... looked up in a profiling database") ----
 * Process-wide map from a block signature (kernel family | operators | data types | shape) to a measured
 * latency in microseconds.  dnnf_plan asks it for the cost of every candidate block of a yellow
 * (profile-dependent) Table 3 decision and of block merging; what it does not find is costed by the
 * analytic model and remembered in the graph as a miss.  All strings are host pointers, NUL-terminated. */
DNNF_API int dnnf_profile_db_set(const char* signature, double microseconds);
DNNF_API int dnnf_profile_db_get(const char* signature, double* microseconds);   /* DNNF_ERR_INVALID_ARG if absent */
DNNF_API int dnnf_profile_db_size(size_t* n_entries);
DNNF_API int dnnf_profile_db_clear(void);
/* Text file, one "signature<TAB>microseconds" line per entry; load adds to / overwrites the current entries. */
DNNF_API int dnnf_profile_db_save(const char* path);
DNNF_API int dnnf_profile_db_load(const char* path, int* n_loaded);
/* Signature of a planned block, and of the i-th miss of the last dnnf_plan (capacity bytes, truncated). */
DNNF_API int dnnf_block_signature(const dnnf_graph* g, int block, char* host_buf, size_t capacity);
DNNF_API int dnnf_profile_miss_count(const dnnf_graph* g, int* n);
DNNF_API int dnnf_profile_miss(const dnnf_graph* g, int index, char* host_buf, size_t capacity);
/* Runs every missed candidate block of the last dnnf_plan on the device and stores its per-launch time in the
 * database: `iters` back-to-back launches between two CUDA events on `cuda_stream`, best of three, after two
 * warm-up launches.  The block's
 * tensors are placed in `scratch` (device memory, 256-byte aligned, contents irrelevant and overwritten);
 * candidates that need more than scratch_bytes are skipped.  Synchronises the stream.  n_measured may be NULL. */
DNNF_API int dnnf_profile_measure(dnnf_graph* g, void* scratch, size_t scratch_bytes, void* cuda_stream, int iters, int* n_measured);

/* ---- binding and execution (Section 4.4: one generated kernel per block) -------- */

/* Bytes of caller-provided device workspace the plan needs for intermediates
 * that stay materialised between blocks plus a small status area. */
DNNF_API int dnnf_workspace_size(const dnnf_graph* g, size_t* bytes);
/* dev_ptr: device memory of the tensor's full size, 16-byte aligned, caller-owned. */
DNNF_API int dnnf_bind(dnnf_graph* g, int tensor_id, void* dev_ptr);
/* The first *bytes of the workspace (status words, then arrival counters of split-K GEMM blocks;
 * at least 256) must be zero when a run starts.  A run that returns DNNF_OK leaves them zero; after
 * a failed run (dnnf_status != DNNF_OK) the caller clears them again. */
DNNF_API int dnnf_workspace_zero_bytes(const dnnf_graph* g, size_t* bytes);
/* dev_ptr: device memory, 256-byte aligned, at least dnnf_workspace_size bytes, its first
 * dnnf_workspace_zero_bytes bytes zero. */
DNNF_API int dnnf_bind_workspace(dnnf_graph* g, void* dev_ptr, size_t bytes);
/* Launches every block's kernel in topological order on `cuda_stream`
 * (a cudaStream_t; NULL = default stream).  Asynchronous. */
DNNF_API int dnnf_run(dnnf_graph* g, void* cuda_stream);
/* Launches only block `block` (for per-block timing). */
DNNF_API int dnnf_run_block(dnnf_graph* g, int block, void* cuda_stream);
/* No counterpart in the paper: a convenience for callers that cannot allocate.
 * Same as dnnf_run(), but the intermediates that stay materialised between blocks
 * live in a fixed array inside the library instead of a caller-provided workspace,
 * so nothing has to be allocated or bound (a workspace bound earlier is ignored for
 * this call and left bound).  Meant for code running where cudaMalloc is off limits:
 * inside a memory pool's out-of-memory handler, in a plugin whose host forbids
 * allocation after initialisation, or between the capture-begin and capture-end of
 * somebody else's stream.
 *  - The array is DNNF_STATIC_WS_BYTES long and is reserved on every GPU that loads
 *    the library, until the process exits.  A plan that needs more returns
 *    DNNF_ERR_WORKSPACE and launches nothing.
 *  - The first call on each device looks the array's address up (with that device
 *    current); make that first call outside any stream capture.
 *  - All graphs and all calls share the one array.  It keeps whatever the previous call
 *    left; the status words at its start are cleared on `cuda_stream` before the
 *    kernels run.  Two calls whose kernels can overlap on the GPU (different streams,
 *    no ordering between them) race on it.
 *  - Inputs and outputs are still the caller's bound tensors.  The call allocates
 *    nothing on host-visible CUDA paths: no cudaMalloc, cudaFree or library routine
 *    that allocates. */
#define DNNF_STATIC_WS_BYTES (32u << 20)
DNNF_API int dnnf_run_static_ws(dnnf_graph* g, void* cuda_stream);
/* After the caller synchronised the stream: device-side status word
 * (0 = ok, DNNF_ERR_TIMEOUT if a bounded wait inside a kernel ran out) and the
 * block that reported it. */
DNNF_API int dnnf_status(dnnf_graph* g, int* device_status, int* block);
/* Self-test of the failure path (no counterpart in the paper).  Every wait inside the tensor-core kernels is bounded;
 * when a bound runs out the kernel records DNNF_ERR_TIMEOUT in the workspace's status words and returns instead of
 * hanging.  This call launches one tiny kernel on `cuda_stream` that waits, with the kernels' own wait routine, on a
 * barrier nobody signals, for at most limit_ns (1 .. 100,000,000).  After a stream synchronisation dnnf_status()
 * reports DNNF_ERR_TIMEOUT from block -2; the caller then clears the workspace's first dnnf_workspace_zero_bytes bytes
 * and the graph runs as before.  Needs a bound workspace; nothing faults, traps or hangs. */
DNNF_API int dnnf_selftest_wait_expiry(dnnf_graph* g, uint64_t limit_ns, void* cuda_stream);
/* Number of kernels one dnnf_run launches. */
DNNF_API int dnnf_launch_count(const dnnf_graph* g, int* n);

DNNF_API const char* dnnf_last_error(const dnnf_graph* g);
DNNF_API const char* dnnf_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DNNF_H_ */
