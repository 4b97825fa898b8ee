/*
 * ago.h -- C ABI of the B200 fused-subgraph executor.
 *
 * A subgraph is an ordered list of operators with shapes (Section II: a
 * computational graph whose nodes are operators and whose edges are tensors;
 * Section III-A, the convolution / bias / ReLU mini-subgraph).
 * Operator i consumes the output of operator i-1; operator 0 consumes
 * subgraph input 0. Operators are either COMPLEX (they reduce: convolution,
 * matrix multiplication) or SIMPLE (element-wise or row-wise: bias, ReLU, add,
 * ...), the split of Section I.
 *
 * Three execution modes:
 *   FUSED              one kernel for the whole subgraph; intermediates stay in
 *                      shared memory / tensor memory (intensive operator
 *                      fusion, Section III-B).
 *   PER_MINI_SUBGRAPH  one kernel per complex operator with its trailing simple
 *                      operators applied in the epilogue (conventional fusion,
 *                      Section III-A, Fig. "Conventional fusion within a
 *                      mini-subgraph"); intermediates round-trip device memory.
 *   PER_OP             one kernel per operator (Section III-A, Fig. "Loop nest
 *                      of a mini-subgraph without fusion").
 *
 * All pointers passed to ago_subgraph_run are DEVICE pointers owned by the
 * caller; the arrays of pointers themselves are host arrays. The library
 * allocates no device memory except one 4-byte status word per handle (at the
 * first run). No call throws or aborts; failures are status codes plus a
 * thread-local message (ago_last_error). There is no CPU fallback: without a
 * CUDA device every run returns AGO_ERR_CUDA.
 *
 * Layouts (row-major, innermost last, 0-based):
 *   activations        NHWC
 *   CONV2D weight      OHWI  [O][R][S][I]; depthwise (groups == C): [R][S][C]
 *   GEMM weight        [K][N]
 *   attention Q,K,V,O  [B][S][heads*head_dim], head h at columns h*D..h*D+D-1
 *   bias vectors       float32 [last dimension]
 * bf16 tensors are raw 16-bit patterns. Every base pointer must be 16-byte
 * aligned (AGO_ERR_ALIGNMENT otherwise).
 */
#ifndef AGO_H_
#define AGO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ago_subgraph_s* ago_subgraph_t; /* opaque; owned by the library */

typedef enum {
  AGO_OK = 0,
  AGO_ERR_INVALID_ARG = 1, /* NULL pointer, bad enum value, bad struct_size          */
  AGO_ERR_UNSUPPORTED = 2, /* valid chain, but no kernel for it in the asked mode     */
  AGO_ERR_SHAPE = 3,       /* operator shapes inconsistent                            */
  AGO_ERR_ALIGNMENT = 4,   /* device pointer not 16-byte aligned                      */
  AGO_ERR_WORKSPACE = 5,   /* workspace missing or too small                          */
  AGO_ERR_CUDA = 6,        /* CUDA runtime / driver error (message has the string)    */
  AGO_ERR_TIMEOUT = 7      /* a bounded device-side wait expired (see ago_subgraph_status) */
} ago_status_t;

typedef enum { AGO_BF16 = 0, AGO_FP32 = 1 } ago_dtype_t; /* FP32 I/O: depthwise-only subgraphs */

typedef enum {
  AGO_MODE_FUSED = 0,
  AGO_MODE_PER_MINI_SUBGRAPH = 1,
  AGO_MODE_PER_OP = 2,
  /* The planner decides between FUSED and PER_MINI_SUBGRAPH (Section VI-B: for some pointwise -> pointwise
   * chains the version WITHOUT intensive fusion is the faster one). It fuses unless the chain has no fused
   * kernel, or the round trip of the intermediates through device memory costs less than about a third of the
   * tensor-core time of the contractions (then both modes are bound by the contractions, and two plain GEMM
   * launches stream their operands better than one kernel that keeps the intermediate on chip). The handle then
   * behaves like a handle of the chosen mode (AGO_Q_MODE tells which; workspace rules of that mode apply). */
  AGO_MODE_AUTO = 3
} ago_mode_t;

typedef enum {
  /* complex operators (Section I: they contain a reduction) */
  AGO_OP_CONV2D = 0,      /* p: O, R, S, stride, pad, groups (1, or C for depthwise with O == C) */
  AGO_OP_GEMM = 1,        /* p: N            out[..., n] = sum_k in[..., k] * w[k][n]          */
  AGO_OP_BATCHED_QKT = 2, /* p: input index of K, heads, head_dim   [B,S,E] -> [B,heads,S,S]   */
  AGO_OP_BATCHED_PV = 3,  /* p: input index of V, heads, head_dim   [B,heads,S,S] -> [B,S,E]   */
  /* simple operators */
  AGO_OP_BIAS_ADD = 4,    /* + float32 vector over the last dimension (consumes one weight)   */
  AGO_OP_RELU = 5,        /* max(x, 0)                                                        */
  AGO_OP_RELU6 = 6,       /* min(max(x, 0), 6)                                                */
  AGO_OP_GELU_TANH = 7,   /* 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))                  */
  AGO_OP_SCALE = 8,       /* x * f                                                            */
  AGO_OP_SOFTMAX_ROWS = 9,/* softmax over the last dimension                                  */
  AGO_OP_ADD_INPUT = 10,  /* p: input index; + that subgraph input, element-wise (residual)   */
  /* layout operators (the reshape / transpose runs of attention blocks, Section VI-B) */
  AGO_OP_RESHAPE = 11,    /* p: rank, d0..d3; same elements in row-major order under a new shape
                             with the same last dimension: a view, never a launch               */
  AGO_OP_TRANSPOSE = 12   /* p: axis a, axis b (neither the last): swap two leading dimensions  */
} ago_op_kind_t;

typedef struct {
  int32_t kind;  /* ago_op_kind_t */
  int32_t p[8];  /* per-kind integer parameters, in the order listed above; rest 0 */
  float f;       /* AGO_OP_SCALE factor */
} ago_op_t;

#define AGO_MAX_INPUTS 4
#define AGO_MAX_RANK 4
#define AGO_MAX_OPS 32

typedef struct {
  uint32_t struct_size;                          /* sizeof(ago_subgraph_desc_t), ABI check */
  int32_t mode;                                  /* ago_mode_t */
  int32_t num_inputs;                            /* 1..AGO_MAX_INPUTS */
  int32_t input_rank[AGO_MAX_INPUTS];            /* 2..4 */
  int64_t input_shape[AGO_MAX_INPUTS][AGO_MAX_RANK];
  int32_t input_dtype[AGO_MAX_INPUTS];           /* ago_dtype_t; all inputs share one dtype */
  int32_t num_ops;                               /* 1..AGO_MAX_OPS */
  const ago_op_t* ops;                           /* copied by create; caller keeps ownership */
  int32_t output_dtype;                          /* ago_dtype_t; must equal the input dtype */
} ago_subgraph_desc_t;

/* What ago_subgraph_query can report (all as int64). */
typedef enum {
  AGO_Q_NUM_WEIGHTS = 0,       /* entries expected in weights[]                                   */
  AGO_Q_WEIGHT_BYTES = 1,      /* + index i in the high half: see AGO_Q_INDEXED                    */
  AGO_Q_OUTPUT_RANK = 2,
  AGO_Q_OUTPUT_DIM = 3,        /* indexed                                                          */
  AGO_Q_OUTPUT_BYTES = 4,
  AGO_Q_FLOPS_TENSOR = 5,      /* 2 * MACs of the dense contractions, as the operators define them */
  AGO_Q_FLOPS_CUDA = 6,        /* 2 * MACs of depthwise convolutions                               */
  AGO_Q_SFU_OPS = 7,           /* exp / tanh evaluations                                           */
  AGO_Q_IO_BYTES = 8,          /* inputs + weights + output; no intermediates                      */
  AGO_Q_NUM_LINKS = 9,         /* adjacent complex -> complex pairs                                */
  AGO_Q_LINK_CATEGORY = 10,    /* indexed; ago_link_category_t                                     */
  AGO_Q_NUM_LAUNCHES = 11,     /* kernels launched by one ago_subgraph_run in this handle's mode   */
  AGO_Q_FUSED_KERNEL = 12,     /* ago_fused_kernel_t chosen by the planner (0 when not fused)      */
  AGO_Q_INTERMEDIATE_BYTES = 13,/* bytes written + read for intermediates in PER_MINI_SUBGRAPH mode */
  AGO_Q_TILE_ROWS = 14,        /* fused kernel: downstream tile extent along the tiled dimension   */
  AGO_Q_SMEM_BYTES = 15,       /* fused kernel: dynamic shared memory per CTA                      */
  AGO_Q_MODE = 16,             /* the mode the handle runs in (what AGO_MODE_AUTO resolved to)     */
  AGO_Q_WORKSPACE_TRAFFIC = 17 /* fused kernel: bytes per run stored or added into / read back from */
                               /* its device-memory workspace (partial sums of a split reduction); not */
                               /* part of AGO_Q_IO_BYTES; 0 when all intermediates stay on chip     */
} ago_query_t;
#define AGO_Q_INDEXED(what, i) ((int32_t)(what) | ((int32_t)(i) << 16))

/* Fusion category of a complex -> complex link (Section III-B, "Removing the
 * Re-computation" and Fig. "Inter-operator data dependency in intensive fusion"). */
typedef enum {
  AGO_LINK_DOWNSTREAM_DEPTHWISE = 1, /* downstream tile H2 W2 o2: spatial dims untiled, channels tiled   */
  AGO_LINK_DOWNSTREAM_POINTWISE = 2, /* downstream tile h2 w2 O2: spatial/rows tiled, all output channels;
                                        matrix multiplication counts as pointwise                       */
  AGO_LINK_GENERAL = 3               /* reuse on O2, H2, W2: fusion needs halo recomputation             */
} ago_link_category_t;

typedef enum {
  AGO_KERNEL_NONE = 0,
  AGO_KERNEL_DEPTHWISE = 1,   /* a depthwise-only mini-subgraph                    */
  AGO_KERNEL_MBV2_BLOCK = 2,  /* 1x1 conv -> depthwise 3x3 -> 1x1 conv [+ residual] */
  AGO_KERNEL_FFN = 3,         /* GEMM -> GELU -> GEMM                               */
  AGO_KERNEL_CONV3X3_PAIR = 4,/* conv3x3 -> conv3x3 [+ residual, ReLU]              */
  AGO_KERNEL_ATTENTION = 5,   /* QK^T -> scale -> softmax -> .V                     */
  /* the two-complex-operator pairs of the fusion-strategy micro-benchmark (Section VI-B) */
  AGO_KERNEL_PW_DW = 6,       /* 1x1 conv -> depthwise 3x3                           */
  AGO_KERNEL_DW_PW = 7,       /* depthwise 3x3 -> 1x1 conv                           */
  AGO_KERNEL_DW_DW = 8,       /* depthwise 3x3 -> depthwise 3x3                      */
  AGO_KERNEL_PW_PW = 9,       /* 1x1 conv -> 1x1 conv                                */
  AGO_KERNEL_GEMM_PERMUTE_GEMM = 10 /* GEMM -> + input -> row transpose -> GEMM (reshapes in between) */
} ago_fused_kernel_t;

/* Validate the operator list, infer shapes, classify every complex -> complex
 * link into the categories of Section III-B and pick the kernels for the asked
 * mode. Host only; no device work. Returns NULL on failure (ago_last_error
 * tells why). The desc and its ops array are copied.
 * FUSED mode serves the chains that have a kernel (ago_fused_kernel_t; query
 * AGO_Q_FUSED_KERNEL) and fails with AGO_ERR_UNSUPPORTED on any other chain or
 * on shapes outside a kernel's limits -- there is no silent fallback:
 *   CONV1x1 BIAS RELU6 DW3x3 BIAS RELU6 CONV1x1 BIAS [ADD_INPUT 0]   inverted residual
 *   CONV1x1 BIAS RELU6 DW3x3 BIAS RELU6 / DW3x3 BIAS RELU6 CONV1x1 BIAS /
 *   DW3x3 BIAS RELU6 DW3x3 BIAS RELU6 (stride 1) /
 *   CONV1x1 BIAS [RELU6] CONV1x1 BIAS [RELU6]                        the pairs of Section VI-B
 *   GEMM BIAS GELU GEMM BIAS                                         feed-forward chain
 *   CONV3x3 BIAS RELU CONV3x3 BIAS ADD_INPUT 0 RELU                  residual 3x3 pair
 *   QKT SCALE SOFTMAX PV                                             attention (head_dim 64,
 *                                   32..384 keys, scale > 0)
 *   GEMM RESHAPE ADD_INPUT RESHAPE TRANSPOSE RESHAPE GEMM RESHAPE    projection chain of a
 *                                   patch-unfolded attention block (rows permuted between the GEMMs)
 *   DW (any window) followed by simple operators only                depthwise mini-subgraph
 * (DW3x3: depthwise, 3x3 window, pad 1, stride 1 or 2). */
ago_subgraph_t ago_subgraph_create(const ago_subgraph_desc_t* desc);

/* Enqueue the subgraph on `cuda_stream` (a cudaStream_t; NULL = the legacy
 * default stream) and return without synchronising.
 *   inputs[num_inputs]  device pointers, in desc order (attention: Q, K, V)
 *   weights[num_weights] device pointers, in order of appearance in the op
 *                        list: each CONV2D / GEMM weight and each BIAS_ADD vector
 *   outputs[1]          device pointer to the result
 * FUSED mode launches one kernel (Section III-B, Fig. "Intensive fusion program
 * of two convolutions": the upstream tile is produced inside the downstream
 * operator's outer tile loops); the unfused modes launch one kernel per
 * operator / per mini-subgraph and need a workspace (ago_subgraph_set_workspace).
 * Errors: AGO_ERR_INVALID_ARG (NULL), AGO_ERR_ALIGNMENT, AGO_ERR_WORKSPACE,
 * AGO_ERR_CUDA (launch failure). */
ago_status_t ago_subgraph_run(ago_subgraph_t h, const void* const* inputs,
                              const void* const* weights, void* const* outputs,
                              void* cuda_stream);

/* Same as ago_subgraph_run, but inputs and the output live in HOST memory
 * (pinned memory makes the copies asynchronous). Per call: copy each host input
 * to the caller's device staging buffer dev_inputs[i], run, copy dev_outputs[0]
 * to host_outputs[0]; all on `cuda_stream`, no synchronisation. Weights stay
 * device pointers. The staging buffers are caller-owned device memory of the
 * tensors' sizes. */
ago_status_t ago_subgraph_run_host(ago_subgraph_t h, const void* const* host_inputs,
                                   const void* const* weights, void* const* host_outputs,
                                   void* const* dev_inputs, void* const* dev_outputs,
                                   void* cuda_stream);

void ago_subgraph_destroy(ago_subgraph_t h); /* NULL is a no-op */

/* Thread-local status and message of the last failing call on this thread. */
ago_status_t ago_last_error(const char** msg);

/* Device workspace for intermediates (unfused modes; 0 for fused kernels that
 * need none). The caller allocates at least ago_subgraph_workspace_bytes(h)
 * bytes, 256-byte aligned, and keeps them alive while the handle is used.
 * The workspace is EXCLUSIVE to the handle between set_workspace and the last
 * run that uses it: a fused kernel that reduces through it (the feed-forward
 * chain at small row counts) zeroes it at the first run after each
 * set_workspace and relies on finding it as it left it afterwards. A caller
 * that lent the buffer to anything else, or whose run failed midway, calls
 * set_workspace again (same pointer is fine) before the next run. */
size_t ago_subgraph_workspace_bytes(ago_subgraph_t h);
ago_status_t ago_subgraph_set_workspace(ago_subgraph_t h, void* dev_ptr, size_t bytes);

/* Plan and work counters; `what` is an ago_query_t, optionally AGO_Q_INDEXED. */
ago_status_t ago_subgraph_query(ago_subgraph_t h, int32_t what, int64_t* out);

/* Synchronises the device and reads the handle's status word: AGO_OK, or
 * AGO_ERR_TIMEOUT when a kernel gave up a bounded wait (its output is then
 * undefined). The word is cleared by the call. */
ago_status_t ago_subgraph_status(ago_subgraph_t h);

/* Test hook for the failure path (Section II, last paragraph, and Section IV
 * "Acyclic Partitioning": the run-time failure the paper names is a wait that
 * never ends, a deadlock between subgraphs that depend on each other; on the
 * device its counterpart is a wait on a signal that never comes). Every
 * device-side wait of this library is bounded; this call lets a test make one
 * run out on a tiny problem without faulting, trapping or hanging the GPU:
 *   AGO_DEBUG_WAIT_BUDGET_US  value = budget of every bounded wait of this
 *                             handle's kernels in microseconds (0 = default, 1 s)
 *   AGO_DEBUG_SKIP_SIGNAL     value = code of a wait site whose producer skips
 *                             its signal (an mbarrier arrival) in every run
 *                             until the value is set back to 0. Sites that
 *                             honour it: 0x104 (fused inverted-residual block:
 *                             "all project MMAs complete"), 0x503 (tensor-core
 *                             GEMM of the unfused modes: "accumulator complete")
 * The waiter gives up after the budget, the kernel runs to its end (output
 * undefined), frees its tensor memory, and ago_subgraph_status returns
 * AGO_ERR_TIMEOUT with the site code in the message. Synchronises the device
 * when the handle has already run. Errors: AGO_ERR_INVALID_ARG. */
typedef enum { AGO_DEBUG_WAIT_BUDGET_US = 1, AGO_DEBUG_SKIP_SIGNAL = 2 } ago_debug_t;
ago_status_t ago_subgraph_debug(ago_subgraph_t h, int32_t what, int64_t value);

/* Bytes of scratch built into the library for ago_subgraph_run_static. */
#define AGO_STATIC_SCRATCH_BYTES (4u << 20)

/* (The paper has no counterpart for this entry point; it exists for deployment.)
 * ago_subgraph_run for PER_OP / PER_MINI_SUBGRAPH handles when nobody may
 * allocate device memory: code that runs inside a host whose memory pools are
 * fixed before it is called (an inference server's plug-in slot, a sandbox that
 * forbids cudaMalloc after start-up, a real-time loop where an allocation's
 * implicit synchronisation is not acceptable). Inputs, weights and the output
 * are still the caller's device buffers; the tensors passed between the
 * launches go to a fixed AGO_STATIC_SCRATCH_BYTES (4 MiB) array inside the
 * library image, which every GPU that loads the library keeps until the
 * process exits. The call allocates and frees nothing, does not use
 * ago_subgraph_set_workspace and does not touch the handle's status word, so
 * a bounded device-side wait that gives up in one of these launches goes
 * unreported (ago_subgraph_status stays AGO_OK).
 *   - A subgraph whose ago_subgraph_workspace_bytes() exceeds the array is
 *     rejected with AGO_ERR_WORKSPACE (message states both sizes); FUSED handles
 *     are rejected with AGO_ERR_UNSUPPORTED (they need no scratch).
 *   - The first call on each device looks up the array's device address (with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on one GPU share the one array, and it keeps the previous
 *     call's contents. Nothing in it has to start at zero (every intermediate is
 *     written in full before it is read), but two calls whose kernels overlap on
 *     the GPU (different streams, different handles or threads) race on it: keep
 *     calls on one stream, or order them with events. */
ago_status_t ago_subgraph_run_static(ago_subgraph_t h, const void* const* inputs,
                                     const void* const* weights, void* const* outputs,
                                     void* cuda_stream);

/* ---- Redundancy of intensive fusion (Section III-B, the GS / TS analysis) -----------------
 * Two stacked convolutions (stride-1 upstream producing [N, O1, H1, W1]; downstream with an
 * R2 x C2 window and stride `stride2` producing [N, O2, H2, W2], windows without padding, so
 * H1 = (H2 - 1) * stride2 + R2 and likewise W1). After tiling the downstream output into tiles
 * of (o2, h2, w2) and fusing, the upstream tile that each downstream tile needs is computed
 * inside the downstream tile loops; an upstream element needed by several downstream tiles is
 * computed once per tile. The call returns how many upstream output elements (and reduction-body
 * executions, x I1 R1 C1) are computed with and without fusion, i.e. the paper's
 * |GS2/TS2 x (GS1/TS1 - GS2/TS2)| * |TS1| against |GS1|, with ragged edge tiles counted exactly.
 * A dense downstream operator (depthwise2 == 0) needs all O1 upstream channels for every tile of
 * output channels; a depthwise one (depthwise2 != 0, O2 == O1) needs the tile's own channels.
 * Tile extents are clamped to the tensor extents. Host-only; no device is touched.
 * Errors: AGO_ERR_INVALID_ARG for NULL pointers, a wrong struct_size or non-positive extents;
 * AGO_ERR_SHAPE when depthwise2 is set and O2 != O1. */
typedef struct {
  uint32_t struct_size;
  int32_t  depthwise2;            /* downstream operator is depthwise (channel c reads upstream channel c) */
  int64_t  N;
  int64_t  O1, I1, R1, C1;        /* upstream: output channels; reduction extents (input channels, window) */
  int64_t  O2, R2, C2, stride2;   /* downstream: output channels, window, stride */
  int64_t  H2, W2;                /* downstream output extent */
  int64_t  o2, h2, w2;            /* downstream tile */
} ago_redundancy_query_t;

typedef struct {
  int64_t num_tiles;              /* downstream tiles = |GS2 / TS2| */
  int64_t upstream_elems_unfused; /* N O1 H1 W1 */
  int64_t upstream_elems_fused;   /* sum over the downstream tiles of the upstream tile each one needs */
  int64_t upstream_macs_unfused;  /* x I1 R1 C1 */
  int64_t upstream_macs_fused;
  double  factor;                 /* fused / unfused; 1.0 = no recomputation */
  int32_t category;               /* ago_link_category_t of the pair */
  int32_t reserved;
} ago_redundancy_result_t;

ago_status_t ago_fusion_redundancy(const ago_redundancy_query_t* q, ago_redundancy_result_t* out);

/* ---- Graph partitioning of the frontend (Section IV, Eq. 1 and Algorithm 1) ----------------
 * Host-only. ago_op_weight is Eq. 1: c * prod over the operator's loops of log(extent) + b
 * (natural logarithm; the paper prints no values for c and b, they are the caller's).
 *
 * ago_graph_cluster runs Algorithm 1 ("Cluster") on a DAG of num_nodes operators with the given
 * weights and num_edges directed edges (edges[2e] -> edges[2e + 1]): repeatedly the heaviest
 * candidate (hyper) node v absorbs the lightest node u of its affix set (adjacent to v, exactly
 * one topological stage above or below, Definitions 2 and 3) while w_v + w_u < threshold, else v
 * leaves the candidates; stages and edges are updated after every merge. By Theorem 1 the
 * resulting partition is acyclic. Ties: heavier first, then the smaller smallest-member id;
 * lighter first, then the smaller smallest-member id.
 * Output: subgraph_of_node[num_nodes] (subgraphs numbered by their smallest member) and
 * *num_subgraphs. Errors: AGO_ERR_INVALID_ARG for NULL arguments, a wrong struct_size, an empty
 * graph, an edge that names no node or a self loop, or a cyclic input graph. */
typedef struct {
  uint32_t struct_size;
  int32_t  num_nodes;
  const double*  weights;   /* [num_nodes] */
  int32_t  num_edges;
  int32_t  reserved;
  const int32_t* edges;     /* [2 * num_edges] */
  double   threshold;       /* Td: a merged subgraph's weight stays below it */
} ago_graph_desc_t;

double       ago_op_weight(const int64_t* loop_extents, int32_t num_loops, double c, double b);
ago_status_t ago_graph_cluster(const ago_graph_desc_t* g, int32_t* subgraph_of_node, int32_t* num_subgraphs);

/* Enqueue a kernel of `grid` CTAs x `block` threads that does nothing, launched the way the fused kernels are
 * (programmatic stream serialization, dynamic shared memory `smem_bytes`): the launch floor against which the
 * launch-bound configurations are read. No device memory is touched. Errors: AGO_ERR_INVALID_ARG for sizes
 * outside 1..65535 CTAs / 1..1024 threads / 0..227 KB, AGO_ERR_CUDA for a failed launch. */
ago_status_t ago_launch_empty(int32_t grid, int32_t block, int32_t smem_bytes, void* cuda_stream);

/* Library version, "major.minor". */
const char* ago_version(void);

#ifdef __cplusplus
}
#endif
#endif /* AGO_H_ */
