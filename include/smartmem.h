/*
 * smartmem.h -- C ABI of the layout-transformation-elimination hot path.
 *
 * The method (SmartMem, ASPLOS '24) removes Reshape / Transpose / Slice / Gather-class
 * operators ("Fixed output" operators, Table 3) from a transformer operator chain by
 * replacing them with index computation inside the operator they are fused with
 * (Section 3.2.1, "Operator Elimination based on Index Comprehension"), after reducing the
 * index arithmetic to its cheapest form (Section 3.2.1, "Strength reduction on index
 * computation").  This library does that for linear operator chains on one B200:
 *
 *   smartmem_plan        host-only planner: operator chain + tensor layouts -> kernel steps,
 *                        each with composed, strength-reduced index maps
 *   smartmem_run_chain   runs a planned chain on a CUDA stream
 *   smartmem_swin_block  one Swin Transformer block (shifted-window attention + MLP)
 *   smartmem_attn_layer  one decoder attention layer (RMSNorm, QKV, RoPE, causal attention, o_proj)
 *
 * Every entry point takes a `mode`: SMARTMEM_ELIMINATE folds all layout operators into the
 * operand loads / result stores of the compute kernels; SMARTMEM_EXPLICIT runs the same
 * compute kernels but materialises every data-moving layout operator with a copy kernel, so
 * the gain from elimination can be measured.
 *
 * Conventions
 *   - All data pointers are DEVICE pointers owned by the caller unless a comment says "host".
 *     The library never allocates device memory; scratch comes from the caller's workspace.
 *   - Tensors are row-major (last dimension contiguous) unless strides are given.  Linear
 *     weights are [out_features, in_features]: the reduction dimension is the contiguous
 *     one for both GEMM operands (Section 3.2.2, reduction-dimension layout rule).
 *   - Calls validate on the host, enqueue work on the given stream and return without
 *     synchronising.  The return value is a smartmem_status_t.  Nothing aborts or prints.
 *   - Device-side waits are bounded; a wait that runs out sets a device status word that
 *     smartmem_last_device_status() reads back.
 *   - There is no CPU fallback: without a CUDA device the run entry points return
 *     SMARTMEM_ERR_CUDA.
 */
#ifndef SMARTMEM_H_
#define SMARTMEM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SMARTMEM_OK = 0,
  SMARTMEM_ERR_INVALID_ARG = -1, /* null pointer, bad enum, bad count                    */
  SMARTMEM_ERR_SHAPE = -2,       /* shapes inconsistent with the operator                */
  SMARTMEM_ERR_UNSUPPORTED = -3, /* valid request the kernels do not cover               */
  SMARTMEM_ERR_WORKSPACE = -4,   /* workspace too small                                  */
  SMARTMEM_ERR_ALIGNMENT = -5,   /* a base pointer is not 16-byte aligned                */
  SMARTMEM_ERR_CUDA = -6,        /* a CUDA runtime/driver call failed (or no device)     */
  SMARTMEM_ERR_TIMEOUT = -7      /* a bounded device-side wait ran out                   */
} smartmem_status_t;

typedef enum { SMARTMEM_F32 = 0, SMARTMEM_BF16 = 1 } smartmem_dtype_t;
/* ELIMINATE_NAIVE (smartmem_plan / smartmem_run_chain only): layout runs are eliminated, but copy
 * consumers evaluate the sequential divide/modulo program instead of the strength-reduced map --
 * the "index computation (no opt.)" form of Fig. 4, kept to measure what strength reduction buys. */
/* ELIMINATE_GATHER / ELIMINATE_SCATTER (smartmem_plan / smartmem_run_chain, copy-only chains of invertible
 * layout operators): the eliminated map is placed on the consumer side (out[i] = in[map(i)]: sub-optimal
 * read, contiguous write) or on the producer side (out[imap(i)] = in[i], imap = the map of the inverted
 * chain: contiguous read, sub-optimal write), both with the plain map-driven kernel -- the two
 * placements Section 3.2.2 compares.  Same result as ELIMINATE, bit for bit. */
/* ELIMINATE_UNFUSED (smartmem_swin_block only): the eliminated chain run kernel by kernel -- LayerNorm + gather +
 * QKV, window attention, projection + scatter + residual, MLP -- each reading its producer's buffer through the
 * composed map.  ELIMINATE additionally fuses the attention half of a narrow block into one kernel (Section 3.2.1:
 * elimination is what makes the fusion possible; Table 5's "try fuse").  Kept so that the two gains are measured apart,
 * and because it runs exactly the arithmetic of EXPLICIT (bit-identical results).  Wide blocks: same as ELIMINATE. */
typedef enum { SMARTMEM_ELIMINATE = 0, SMARTMEM_EXPLICIT = 1, SMARTMEM_ELIMINATE_NAIVE = 2,
               SMARTMEM_ELIMINATE_GATHER = 3, SMARTMEM_ELIMINATE_SCATTER = 4, SMARTMEM_ELIMINATE_UNFUSED = 5 } smartmem_mode_t;

/* Operator vocabulary of a chain.  Layout operators have a Fixed output layout (Table 3,
 * right column) and are the ones elimination removes; compute operators are kept. */
typedef enum {
  SMARTMEM_OP_RESHAPE = 0,          /* shape[] = new shape                                 */
  SMARTMEM_OP_TRANSPOSE = 1,        /* perm[]: out.shape[k] = in.shape[perm[k]]            */
  SMARTMEM_OP_ROLL = 2,             /* axis, shift[0]: out[j] = in[(j - shift) mod N]      */
  SMARTMEM_OP_SLICE = 3,            /* start[], shape[] = extent                           */
  SMARTMEM_OP_WINDOW_PARTITION = 4, /* [B,H,W,C] -> [B*H/ws*W/ws, ws*ws, C]; window = ws   */
  SMARTMEM_OP_WINDOW_REVERSE = 5,   /* inverse; shape[0..2] = B,H,W                        */
  SMARTMEM_OP_DEPTH_TO_SPACE = 6,   /* [N,C*b*b,H,W] -> [N,C,H*b,W*b]: out[n,c,h*b+i,w*b+j] = in[n,(i*b+j)*C+c,h,w]; window = b
                                       (Table 3's DtoS; depth-column-row order)             */
  SMARTMEM_OP_SPACE_TO_DEPTH = 7,   /* inverse (Table 3's StoD): [N,C,H,W] -> [N,C*b*b,H/b,W/b]; window = b */
  SMARTMEM_OP_COPY = 16,            /* consumer: writes the current tensor contiguously    */
  SMARTMEM_OP_LINEAR = 17,          /* consumer: out[M,N] = A[M,K] W[N,K]^T, W = side_input[0] */
  SMARTMEM_OP_BMM_NT = 18,          /* consumer: out[..,i,j] = sum_e A[..,i,e] B[..,j,e]; B is the
                                       result of running the same layout run on side_input[0] */
  SMARTMEM_OP_LAYERNORM = 19        /* consumer: LayerNorm over the last dimension (an ILD & Variable operator of
                                       Table 3): gamma = side_input[0], beta = side_input[1], both [C]; eps   */
} smartmem_op_kind_t;

#define SMARTMEM_MAX_DIMS 8
#define SMARTMEM_MAX_ATOMS 16
#define SMARTMEM_MAX_ROLLS 4

typedef struct {
  int32_t kind;                      /* smartmem_op_kind_t                                  */
  int32_t ndim;                      /* entries used in shape / perm / start                */
  int64_t shape[SMARTMEM_MAX_DIMS];  /* reshape target, slice extent, window_reverse B,H,W  */
  int32_t perm[SMARTMEM_MAX_DIMS];   /* transpose                                           */
  int64_t start[SMARTMEM_MAX_DIMS];  /* slice                                               */
  int64_t shift;                     /* roll                                                */
  int32_t axis;                      /* roll                                                */
  int32_t window;                    /* window partition / reverse; block size of depth/space */
  int32_t side_input[2];             /* index into the plan's inputs[] (weights, 2nd operand) */
  float eps;                         /* layernorm                                           */
  int32_t reserved;                  /* zero                                                */
} smartmem_op_t;

typedef struct {
  int32_t dtype;                     /* smartmem_dtype_t                                    */
  int32_t ndim;
  int64_t shape[SMARTMEM_MAX_DIMS];
  int64_t stride[SMARTMEM_MAX_DIMS]; /* in elements; all zero = contiguous row-major        */
} smartmem_tensor_desc_t;

/* A composed index map in canonical form (Section 3.2.1: identity / split / merge index
 * dependencies derived from static shapes, then strength-reduced).  The consumer's linear
 * index i (row-major over its logical shape) is written in mixed radix over `extent[]`
 * (atom 0 is the most significant digit); the source offset in elements is
 *
 *     base + sum_{a : roll_of[a] < 0} digit_a * src_stride[a]
 *          + sum_r place_r( (sum_{a : roll_of[a] == r} digit_a * roll_weight[a] + roll_shift[r]) mod roll_mod[r] )
 *
 * where place_r(v) = v * roll_stride[r] when the rolled dimension is an affine coordinate of the
 * producer's buffer (roll_n_parts[r] == 1), and otherwise v is written in mixed radix over
 * roll_part_extent[r][] (part 0 most significant) and each digit is multiplied by
 * roll_part_stride[r][] (a dimension rolled after it was merged from non-nesting factors, e.g.
 * H after a window reverse).  No division or modulo by tensor extents survives except one
 * modulo per rolled dimension (and the part digits of such merged dimensions).  klass: 0 identity (the chain vanishes), 1 affine (no roll; a TMA tensor map or
 * a tiled transpose can express it), 2 strided gather with rolls, 3 not canonicalisable
 * (the split points of the shapes do not refine each other): only the sequential
 * divide/modulo program -- the unoptimised form of Fig. 4 -- can evaluate it. */
typedef struct {
  int32_t n_atoms;
  int64_t extent[SMARTMEM_MAX_ATOMS];
  int64_t src_stride[SMARTMEM_MAX_ATOMS];
  int32_t roll_of[SMARTMEM_MAX_ATOMS];
  int64_t roll_weight[SMARTMEM_MAX_ATOMS];
  int32_t n_rolls;
  int64_t roll_shift[SMARTMEM_MAX_ROLLS];
  int64_t roll_mod[SMARTMEM_MAX_ROLLS];
  int64_t roll_stride[SMARTMEM_MAX_ROLLS];
  int32_t roll_n_parts[SMARTMEM_MAX_ROLLS];
  int64_t roll_part_extent[SMARTMEM_MAX_ROLLS][SMARTMEM_MAX_ROLLS];
  int64_t roll_part_stride[SMARTMEM_MAX_ROLLS][SMARTMEM_MAX_ROLLS];
  int64_t base;
  int64_t n_elements;                /* number of consumer elements                         */
  int32_t vec_elems;                 /* widest power-of-two run (<= 16 bytes) that is contiguous
                                        in both source and consumer and never straddles a wrap */
  int32_t klass;
} smartmem_index_map_t;

typedef struct smartmem_plan smartmem_plan_t; /* opaque, library-owned, host memory */

/* Operator classification (Table 3) and the pairwise decisions of Tables 5 and 6.
 * quadrant: 0 ILD&Variable, 1 ILI&Variable, 2 ILD&Fixed, 3 ILI&Fixed.
 * action  : 0 keep both, 1 try fuse, 2 eliminate 1st, 3 eliminate 2nd, 4 eliminate both.
 * result  : resulting quadrant, or -1 where the table says N/A.
 * search  : 0 no search, 1 search both, 2 search fused, 3 search 1st, 4 search 2nd. */
int smartmem_op_quadrant(int32_t op_kind, int32_t* quadrant);
int smartmem_pair_decision(int32_t first_quadrant, int32_t second_quadrant, int32_t* action,
                           int32_t* result, int32_t* search);

/* Reduction-dimension layout selection for a producer with several consumers (Section 3.2.2, "Global:
 * layout selections based on reduction dimension"; host only).  The producer's result has `ndim`
 * dimensions; consumer c aggregates along producer dimension reduction_dim[c] (-1: no requirement) and
 * counts with weight[c] > 0 (null: all 1; e.g. how often it runs or how many bytes it reads).  `k` is
 * the number of memory dimensions that can be walked contiguously without index arithmetic (1 for
 * linear memory, 2 for the paper's 2.5D texture memory).
 *   Layout 0 serves the k most demanded reduction dimensions (demand = summed weight; ties go to the
 * dimension that is already innermost-most): they become its k innermost dimensions, the most demanded
 * one innermost (contiguous); all other dimensions keep their relative order outside.  Consumers whose
 * reduction dimension is not among them are served by further copies of the tensor ("several copies of
 * data with different layouts"), layout 1 taking the next k most demanded dimensions, and so on.
 *   Outputs: *n_layouts; perm[l * SMARTMEM_MAX_DIMS + p] = producer dimension stored at position p of
 * layout l (position 0 outermost, ndim-1 contiguous); layout_of_consumer[c] = the layout consumer c reads
 * (0 for consumers without a requirement).  Errors: INVALID_ARG (null, ndim or k out of range, a
 * reduction dimension >= ndim, weight <= 0), UNSUPPORTED (more than max_layouts layouts needed). */
int smartmem_select_layouts(int32_t ndim, int32_t n_consumers, const int32_t* reduction_dim, const int64_t* weight,
                            int32_t k, int32_t max_layouts, int32_t* n_layouts, int32_t* perm,
                            int32_t* layout_of_consumer);

/* Host only (no CUDA call).  Walks the chain, splits it at compute operators, and for each
 * maximal run of layout operators composes the index map (ELIMINATE) or emits one copy
 * step per data-moving layout operator (EXPLICIT; a Reshape of a contiguous tensor stays
 * metadata).  inputs[0] is the chain's input, other entries are side inputs.
 * Errors: INVALID_ARG, SHAPE (operator/shape mismatch), UNSUPPORTED. */
int smartmem_plan(const smartmem_op_t* ops, int32_t n_ops, const smartmem_tensor_desc_t* inputs,
                  int32_t n_inputs, int32_t mode, smartmem_plan_t** out_plan);
int smartmem_plan_destroy(smartmem_plan_t* plan);
/* Number of kernel steps in total and how many of them are layout copies. */
int smartmem_plan_num_steps(const smartmem_plan_t* plan, int32_t* n_steps, int32_t* n_copies);
/* Index map of operand `operand` (0 = first/A operand, 1 = second/B operand) of step `step`. */
int smartmem_plan_get_map(const smartmem_plan_t* plan, int32_t step, int32_t operand,
                          smartmem_index_map_t* out);
/* Logical shape of the chain's result. */
int smartmem_plan_output_desc(const smartmem_plan_t* plan, smartmem_tensor_desc_t* out);
/* Bytes of device workspace smartmem_run_chain needs (intermediate copies in EXPLICIT mode). */
int smartmem_plan_workspace_bytes(const smartmem_plan_t* plan, size_t* bytes);
/* Host evaluators, for tests: source offset of consumer element i through the canonical map,
 * and through the sequential divide/modulo program of the same run (the unoptimised form). */
int64_t smartmem_map_eval(const smartmem_index_map_t* map, int64_t consumer_linear_index);
int64_t smartmem_plan_eval_sequential(const smartmem_plan_t* plan, int32_t step, int32_t operand,
                                      int64_t consumer_linear_index);

/* Enqueues the plan's kernels.  inputs[i] matches the planner's inputs[i]; outputs[0] receives
 * the result (contiguous, bf16 or f32 as the input dtype).  `cuda_stream` is a cudaStream_t. */
int smartmem_run_chain(const smartmem_plan_t* plan, const void* const* inputs, void* const* outputs,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/* One Swin block.  x, y: [B,H,W,C]; y = x + proj(window_attention(LN1(x))) and, when
 * mlp_ratio > 0, then y += fc2(GELU(fc1(LN2(y)))).  rel_bias_table is [(2*window-1)^2, heads].
 * Requirements: window divides H and W; 0 <= shift < window; C = heads * head_dim with
 * head_dim in {16, 32}; window*window <= 64; x and y must not alias.
 * dtype F32 runs plain-FMA kernels (a 10-bit-mantissa tensor-core path cannot meet 1e-4);
 * dtype BF16 runs the tensor-core kernels with fp32 accumulation, statistics and softmax. */
typedef struct {
  int32_t dtype, B, H, W, C, heads, window, shift, mlp_ratio;
  float ln_eps;
  const void *ln1_g, *ln1_b, *w_qkv, *b_qkv, *rel_bias_table, *w_proj, *b_proj;
  const void *ln2_g, *ln2_b, *w_fc1, *b_fc1, *w_fc2, *b_fc2;
} smartmem_swin_params_t;
int smartmem_swin_block_workspace_bytes(const smartmem_swin_params_t* p, int32_t mode, size_t* bytes);
int smartmem_swin_block(const smartmem_swin_params_t* p, const void* x, void* y, void* workspace,
                        size_t workspace_bytes, int32_t mode, void* cuda_stream);

/* One half of the block on its own (Section 3.2.1's chain splits at the residual between the two halves):
 * half = 0: y = x + proj(attention(LN1(x)))  (the attention half; what mlp_ratio = 0 computes),
 * half = 1: y = x + fc2(GELU(fc1(LN2(x))))   (the MLP half; x is an attention half's result; needs mlp_ratio > 0).
 * Same requirements, modes and workspace size as smartmem_swin_block; running half 0 into a buffer and half 1 from it
 * gives the block's result bit for bit.  Lets a caller place its own work between the halves, and a benchmark time
 * each half back to back. */
int smartmem_swin_block_half(const smartmem_swin_params_t* p, const void* x, void* y, void* workspace,
                             size_t workspace_bytes, int32_t mode, int32_t half, void* cuda_stream);

/* Measurement aid (no counterpart in the paper): the same block, with a CUDA event recorded on
 * `cuda_stream` before every kernel launch.  Synchronises the stream, then writes the duration of
 * each kernel in milliseconds to kernel_ms[i] (host) and its label, NUL-terminated, to
 * kernel_names + i * names_stride (host); *n_kernels receives the count (at most max_kernels). */
int smartmem_swin_block_timed(const smartmem_swin_params_t* p, const void* x, void* y, void* workspace,
                              size_t workspace_bytes, int32_t mode, void* cuda_stream, float* kernel_ms,
                              char* kernel_names, int32_t names_stride, int32_t max_kernels,
                              int32_t* n_kernels);

/* Measurement aid for any entry point (no counterpart in the paper): between smartmem_profile_begin()
 * and smartmem_profile_end() every kernel launch of the library is preceded by a CUDA event on
 * its stream.  _end records a last event on `cuda_stream`, synchronises it and writes each
 * kernel's duration (ms) and label as smartmem_swin_block_timed does.  Not thread-safe against
 * concurrent launches from other host threads; meant for benchmarks. */
int smartmem_profile_begin(void);
int smartmem_profile_end(void* cuda_stream, float* kernel_ms, char* kernel_names, int32_t names_stride,
                         int32_t max_kernels, int32_t* n_kernels);

/* The Swin block for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a deployment aid).  Typical callers: a step that runs while the process's device
 * memory pool is frozen (everything committed to caches and activations, so a cudaMalloc would
 * fail or stall the device), a plugin that is handed buffers and a stream but not the host's
 * allocator, or start-up code that runs before any allocator exists.  They pass only x and y;
 * the block's intermediates go to a fixed array of SMARTMEM_STATIC_SCRATCH bytes (32 MiB,
 * reported by smartmem_swin_block_static_scratch_bytes) that is part of the library image:
 * every GPU that loads the library holds those 32 MiB until the process exits.
 *
 *  - Same arguments, requirements and results as smartmem_swin_block, minus the workspace.
 *  - A block whose intermediates need more than the fixed array (see
 *    smartmem_swin_block_workspace_bytes) is rejected with SMARTMEM_ERR_WORKSPACE
 *    ("workspace too small"); nothing is launched.
 *  - The call itself performs no device allocation and frees nothing: no cudaMalloc / cudaFree and
 *    no allocating library routine.  The first call on each device looks up the array's device
 *    address (the device must be current); make that first call before starting any stream
 *    capture on that device.
 *  - All calls on a device share the one array, and it keeps whatever the previous call left in it.
 *    The block overwrites every intermediate before reading it, so nothing needs clearing; but two
 *    calls whose kernels overlap on the GPU (different streams, no ordering between them) race on
 *    the array and corrupt each other.  Order them on one stream or with events. */
int smartmem_swin_block_static_scratch_bytes(size_t* bytes);
int smartmem_swin_block_noalloc(const smartmem_swin_params_t* p, const void* x, void* y, int32_t mode,
                                void* cuda_stream);

/* One decoder attention layer, prefill.  x, y: [B,S,hidden], bf16.  w_qkv is [3*hidden, hidden]
 * with output columns ordered (q|k|v, head, head_dim); RoPE pairs (i, i + R/2) over the first R =
 * rotary_dim columns of every head at frequencies theta^(-2i/R), the other columns pass unrotated
 * (rotary_dim 0 means head_dim: the whole head rotates; 32 and 64 are the partial-rotary layers of
 * the Pythia / GPT-NeoX family, which the paper's evaluation includes). */
typedef struct {
  int32_t dtype, B, S, hidden, heads, head_dim, causal, add_residual;
  float rms_eps, rope_theta;
  const void *rms_g, *w_qkv, *w_o;
  int32_t rotary_dim;                /* 0 (= head_dim), 32, 64 or 128 */
  int32_t reserved;                  /* zero */
} smartmem_attn_params_t;
int smartmem_attn_layer_workspace_bytes(const smartmem_attn_params_t* p, int32_t mode, size_t* bytes);
int smartmem_attn_layer(const smartmem_attn_params_t* p, const void* x, void* y, void* workspace,
                        size_t workspace_bytes, int32_t mode, void* cuda_stream);

/* One decode step of the same layer against a key/value cache (the decode-time form of the chain
 * of Section 2 / Fig. 1: the Concat that appends the new key and value, the head split and the
 * head merge are Fixed-output layout operators of Table 3 and are eliminated; Section 3.2.2's
 * "sub-optimal write" placement puts the append on the producer's store).
 *
 * B independent sequences, each holding `pos` cached positions (0 <= pos < S_max); the new token of
 * each sits at position pos.  x, y: [B,hidden] bf16 (device), x != y.  p->S is S_max, p->causal is
 * ignored (the last row of a causal mask is all-true), other fields as for smartmem_attn_layer.
 * k_cache, v_cache (device, bf16, 16-byte aligned, owned by the caller, updated in place: row pos
 * of every sequence is written, rows [0,pos) are read, nothing else is touched); keys are stored
 * rotated.  Their layout depends on the mode, because the layout IS the point:
 *   SMARTMEM_ELIMINATE  [B, S_max, heads, head_dim]  -- the layout the QKV GEMM produces: its
 *       epilogue rotates q and k at position pos and stores the k and v columns of row b straight
 *       into cache row (b, pos); attention reads head h as a strided slice and writes its output at
 *       column h*head_dim of [B,hidden].  No copy kernel runs.
 *   SMARTMEM_EXPLICIT   [B, heads, S_max, head_dim]  -- the per-head layout of the materialised
 *       chain: plain QKV GEMM, head-split copy, stand-alone rotary pass, append copy into the cache,
 *       attention on contiguous per-head tensors.
 * head_dim must be 128, hidden a multiple of 256, pos + 1 <= 16384; otherwise
 * SMARTMEM_ERR_UNSUPPORTED.  Errors as for smartmem_attn_layer. */
int smartmem_attn_decode_workspace_bytes(const smartmem_attn_params_t* p, int32_t mode, size_t* bytes);
int smartmem_attn_decode(const smartmem_attn_params_t* p, int32_t pos, const void* x, void* k_cache, void* v_cache,
                         void* y, void* workspace, size_t workspace_bytes, int32_t mode, void* cuda_stream);

/* Synchronises the stream and returns the device status word (SMARTMEM_OK, _TIMEOUT or _UNSUPPORTED)
 * in *status, then clears it. */
int smartmem_last_device_status(void* cuda_stream, int32_t* status);
/* ---- A producer with two consumers of different reduction dimensions (Section 3.2.2, "Global: layout
 * selections based on reduction dimension", and the redundant-copy remark in the discussion of the evaluation).
 *   P  = X Wp^T           X [B*S, K], Wp [N, K]; P is the tensor [B, S, N]
 *   YA = P Wa^T           Wa [Na, N]: aggregates along N (dimension 2 of P);          YA [B*S, Na]
 *   YB[b] = P[b]^T Wb^T   Wb [Nb, S]: aggregates along S (dimension 1 of P);          YB [B, N, Nb]
 * bf16, device pointers, every extent a multiple of 8.  k_contig is the k of smartmem_select_layouts: with
 * k_contig = 2 the planner keeps ONE copy of P in [B, S, N] and consumer B reads it with S as its reduction
 * dimension through a tiled (TMA) operand; with k_contig = 1 it asks for two copies and the producer's epilogue
 * writes [B, S, N] and [B, N, S].  SMARTMEM_EXPLICIT writes [B, S, N] and transposes it with a copy kernel.
 * The three variants give identical YA; YB is identical between k_contig = 1 and EXPLICIT. */
typedef struct {
  int32_t B, S, K, N, Na, Nb;
  int32_t k_contig;                 /* 1 or 2 (ignored by SMARTMEM_EXPLICIT) */
  const void *w_p, *w_a, *w_b;      /* device, bf16 */
} smartmem_fanout_params_t;
/* What the planner decided (host only; any output pointer may be null): copies of P written in total, the layout
 * consumer B reads (0: [B,S,N], 1: [B,N,S]), bytes of P the producer's epilogue writes, bytes the transposing copy
 * kernel moves (EXPLICIT only, read + write), and the workspace the call needs. */
int smartmem_fanout_plan(const smartmem_fanout_params_t* p, int32_t mode, int32_t* n_copies_written,
                         int32_t* layout_of_consumer_b, int64_t* producer_bytes_written, int64_t* copy_kernel_bytes,
                         size_t* workspace_bytes);
/* Runs producer and consumers on the stream.  x, ya, yb and the workspace are device memory owned by the caller
 * (16-byte aligned); nothing is allocated.  Errors: INVALID_ARG (null pointer, extent < 1, mode other than
 * ELIMINATE / EXPLICIT, k_contig outside 1..2), UNSUPPORTED (an extent that is not a multiple of 8), WORKSPACE. */
int smartmem_fanout(const smartmem_fanout_params_t* p, const void* x, void* ya, void* yb, void* workspace,
                    size_t workspace_bytes, int32_t mode, void* cuda_stream);

/* Limit, in nanoseconds, of every bounded device-side wait of the current device (default 1e9, at most 6e10).
 * A wait that runs out makes its kernel unwind and return normally with SMARTMEM_ERR_TIMEOUT in the device
 * status word.  Synchronises the device.  SMARTMEM_ERR_INVALID_ARG for 0 or more than 60 s. */
int smartmem_set_wait_limit_ns(uint64_t limit_ns);
/* Self-test of that unwind: launches one warp that waits, through the kernels' own bounded wait, on a barrier
 * nothing arrives at.  After the wait limit the kernel returns; smartmem_last_device_status() then reports
 * SMARTMEM_ERR_TIMEOUT and the context stays usable.  No memory is touched besides the status word. */
int smartmem_selftest_bounded_wait(void* cuda_stream);
/* Number of kernels this library has launched since it was loaded (for benchmark accounting). */
int64_t smartmem_launch_count(void);
const char* smartmem_status_string(int32_t status);

#ifdef __cplusplus
}
#endif
#endif /* SMARTMEM_H_ */
