/*
 * fluid.h — C-ABI of the planned-arena transformer executor for NVIDIA B200 (sm_100a).
 *
 * The two central calls follow the paper's problem statement (FluidML, Sec. "Design"):
 *   fluid_plan(graph, layout_candidates) -> plan   chooses, on the host, one memory layout per
 *       tensor ("edge") and one offset per activation inside a single shared arena;
 *   fluid_run(plan, arena_ptr, inputs, outputs, stream)   executes that blueprint on the GPU.
 *
 * Conventions for every call
 *   - Return value: FLUID_OK (0) or a negative fluid_status_t; fluid_last_error() gives a
 *     thread-local message for the last failure. Nothing throws or aborts across this boundary.
 *   - Ownership: the caller owns every device byte (arena, inputs, outputs, constants). The
 *     library owns only host memory inside fluid_graph_t / fluid_plan_t objects and never allocates
 *     or frees device memory.
 *   - "dev" pointers are device addresses; everything else is host memory.
 *   - A layout of a rank-r tensor is a permutation of its logical dims listed slowest to
 *     fastest with dense strides; the identity is canonical row-major. For a matrix (0,1) is
 *     row-major and (1,0) column-major (paper, Sec. "Background", Fig. "matmul").
 *   - Graph inputs and outputs are dense canonical buffers, passed in declaration order.
 */
#ifndef FLUID_H
#define FLUID_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define FLUID_API __attribute__((visibility("default")))
#else
#define FLUID_API
#endif

#define FLUID_MAX_RANK 5
#define FLUID_ARENA_ALIGN 1024   /* required alignment of arena_ptr, bytes */
#define FLUID_ARENA_HEADER 256   /* reserved bytes at arena offset 0 (device status words) */
#define FLUID_SLOT_ALIGN 256     /* every planned offset and size is a multiple of this */

typedef struct fluid_graph_s fluid_graph_t; /* host object, opaque, library-owned */
typedef struct fluid_plan_s fluid_plan_t;   /* host object, opaque, library-owned */
typedef void* fluid_stream;             /* a cudaStream_t (NULL = the legacy default stream) */

typedef enum {
  FLUID_OK = 0,
  FLUID_EINVAL = -1,       /* malformed argument, graph or plan */
  FLUID_EUNSUPPORTED = -2, /* no kernel for this op / layout combination (reported at plan time) */
  FLUID_EALIGN = -3,       /* a device pointer is not aligned as required */
  FLUID_ECUDA = -4,        /* a CUDA call or launch failed */
  FLUID_ENOMEM = -5,       /* host allocation failed */
  FLUID_ETIMEOUT = -6      /* a bounded device-side wait expired (see fluid_status) */
} fluid_status_t;

typedef enum { FLUID_F32 = 0, FLUID_BF16 = 1, FLUID_I32 = 2 } fluid_dtype;
/* FLUID_STATE: a caller-owned device buffer that a step both reads and updates and that lives on between runs (a
 * key/value cache). It is passed to fluid_run among `inputs`, in declaration order with the FLUID_INPUT tensors,
 * stays canonical and never sits in the arena. */
typedef enum { FLUID_INPUT = 0, FLUID_OUTPUT = 1, FLUID_CONST = 2, FLUID_ACT = 3, FLUID_STATE = 4 } fluid_tensor_kind;

/* Primitive operators ("nodes"). Shapes are logical, independent of layout.
 *  EMBED   (ids[B,S] i32, tok[V,H] [, pos[P,H] [, off i32[1] or i32[B]]]) -> x[b,s,:] = tok[ids[b,s]] (+ pos[s + off]);
 *          off (read on the device at run time) is the number of tokens that came before, for the batch or per
 *          sequence; ids are clamped to [0,V) and position rows to [0,P)
 *  LINEAR  (x[..m.., ..k..], w[..k.., ..n..] [, bias[..n..]]) -> y[..m.., ..n..]; contracts the
 *          last `contract` dims of x with the first `contract` dims of w (the paper's GEMM:
 *          left (i,k), right (k,j), out (i,j))
 *  ADD, MUL (a, b) -> elementwise, same shape;  GELU, SILU (x) -> elementwise
 *  SOFTMAX (s[..., n]) -> over the last dim, after multiplying by `scale`; causal: column j of
 *          row i (the last two dims) takes part only if j <= i, other outputs are exactly 0
 *  LAYERNORM (x, gamma, beta) / RMSNORM (x, gamma) -> over the last dim, population variance
 *  ROPE    (x[B,S,nh,D] [, pos i32[1] or i32[B]]) -> rotary embedding with position = index along dim 1 (+ pos[0], or
 *          pos[b] per sequence, read on the device at run time: the number of tokens that came before this call's
 *          first row)
 *  TRANSPOSE (x) -> y with y dim j = x dim perm[j]
 *  BMM_QK  (q[B,nh,S,D], kt[B,nh,D,S]) -> scale * q.kt  [B,nh,S,S]
 *  BMM_PV  (p[B,nh,S,S], v[B,nh,S,D]) -> p.v  [B,nh,S,D]
 *  SELECT_LAST_TOKEN (x[B,S,H]) -> x[:, S-1, :]  [B,H]
 *  CACHED_ATTENTION (q[B,1,nh,D], k[B,1,nkv,D], v[B,1,nkv,D], k_cache STATE[B,Tmax,nkv,D], v_cache STATE[B,Tmax,nkv,D],
 *          pos i32[1] or i32[B]) -> ctx[B,1,nh,D]: one decoding step. With t = pos[0] for every sequence, or pos[b]
 *          for sequence b (read on the device at run time, 0 <= t < Tmax) the step stores k, v as row t of the caches and returns
 *          ctx[b,0,h,:] = sum_{j<=t} softmax_j(scale * q[b,0,h,:] . k_cache[b,j,g,:]) v_cache[b,j,g,:], g = h / (nh/nkv):
 *          the row for position t of causal attention over the t+1 tokens so far. Cache rows beyond t are neither
 *          read nor written. t outside [0, Tmax) leaves that sequence's caches and ctx untouched and sets bit 0x10 of
 *          fluid_status.
 */
typedef enum {
  FLUID_OP_EMBED = 0, FLUID_OP_LINEAR = 1, FLUID_OP_ADD = 2, FLUID_OP_MUL = 3, FLUID_OP_GELU = 4,
  FLUID_OP_SILU = 5, FLUID_OP_SOFTMAX = 6, FLUID_OP_LAYERNORM = 7, FLUID_OP_RMSNORM = 8,
  FLUID_OP_ROPE = 9, FLUID_OP_TRANSPOSE = 10, FLUID_OP_BMM_QK = 11, FLUID_OP_BMM_PV = 12,
  FLUID_OP_SELECT_LAST_TOKEN = 13, FLUID_OP_CACHED_ATTENTION = 14, FLUID_OP_COUNT = 15
} fluid_op_kind;

/* One attribute block serves every operator; unused fields are ignored. */
typedef struct fluid_op_attrs {
  int32_t contract;          /* LINEAR: number of contracted dims (>= 1) */
  int32_t causal;            /* SOFTMAX */
  int32_t gelu_tanh;         /* GELU: 0 = erf form, 1 = tanh approximation */
  int32_t rope_interleaved;  /* ROPE: 0 = pairs (i, i+D/2), 1 = pairs (2i, 2i+1) */
  int32_t perm[8];           /* TRANSPOSE */
  double scale;              /* BMM_QK, SOFTMAX, CACHED_ATTENTION (0 is read as 1) */
  double eps;                /* LAYERNORM, RMSNORM */
  double rope_base;          /* ROPE */
} fluid_op_attrs;

/* Layout options per tensor (the paper's L(u): "each with a few diverse memory layout
 * options"). n_cands[t] == 0 means canonical only. perms holds, tensor after tensor, n_cands[t]
 * permutations of rank(t) ints each; the first candidate of a tensor must be the identity. */
typedef struct fluid_layout_candidates {
  int32_t n_tensors;
  const int32_t* n_cands;
  const int32_t* perms;
} fluid_layout_candidates;

/* The paper's external cost function eval(node, layouts) (Algorithm 3): the time of one node
 * given a layout index for each of its tensors. Return +infinity for an unsupported
 * combination. node_id is the graph's op id (custom evaluation implies fusion = 0). If the function
 * rates as finite a combination that no kernel can run and the plan ends up using it, fluid_plan
 * still returns the plan (sequences, layouts and arena can be inspected) and fluid_run refuses it
 * with FLUID_EUNSUPPORTED. */
typedef double (*fluid_eval_fn)(void* user, int32_t node_id, int32_t n_tensors,
                                const int32_t* tensor_ids, const int32_t* layout_index);
typedef double (*fluid_eval_variant_fn)(void* user, int32_t node_id, int32_t n_tensors,
                                        const int32_t* tensor_ids, const int32_t* layout_index, int32_t variant);

typedef struct fluid_plan_options {
  int32_t fusion;           /* 1: fold bias/GELU/residual into GEMM epilogues, residual into norms,
                               SiLU*up into one pass, and BMM_QK -> SOFTMAX -> BMM_PV into one
                               attention step whose score tensor never leaves the SM;
                               0: one step per graph op */
  int32_t arena_policy;     /* 0: first fit (Algorithm 4 as printed), 1: best fit (its prose), 2 (not in the paper): the
                               same placement over several record orders and both fits, the smallest arena kept */
  int32_t no_reuse;         /* 1: one private slice per activation (the naive plan) */
  int32_t force_canonical;  /* 1: skip the layout search, every tensor canonical */
  int32_t gemm_path;        /* 0: tensor cores where eligible, 1: SIMT kernel everywhere */
  int32_t narrow_stream;    /* bf16 graphs: 0 = activations that only feed normalisations and
                               residual additions (the residual stream) are held in fp32 inside the
                               arena, with a bf16 twin where a GEMM also reads them; 1 = every
                               activation is held in its declared dtype */
  int32_t unfused_attention; /* 1: keep BMM_QK -> SOFTMAX -> BMM_PV as three steps even when fusion is on */
  int32_t split_k;          /* GEMM steps with few output tiles cut their k range across CTAs.
                               0 (default): where one thread-block cluster per output tile fits the GPU in one
                               wave, the cut runs inside the cluster and the partial sums meet in distributed
                               shared memory (no scratch; the arena holds activations only).
                               1: in addition, steps with a long k range may park fp32 partial tiles in a scratch
                               slice of the arena that lives for that step.
                               -1: never split */
  fluid_eval_fn eval;       /* NULL: built-in analytic B200 cost table */
  void* eval_user;
  /* Implementation variants (the paper's "Loop Reordering": the time T of a matrix-multiply-like node that the
   * dynamic programme sees is the best over its implementation variants, and that variant is the one that runs).
   * A tensor-core GEMM node has the variants listed by fluid_gemm_variants for its shape and layouts
   * (code = form | tile_n << 4; form 1: one CTA per 128 x tile_n tile, 2: a CTA pair per 256 x tile_n tile (tile_n 256, or 192 for single steps with a k-contiguous weight),
   * 3: a thread-block cluster per tile that splits k). With the built-in table every variant is rated by an analytic
   * model (waves of tiles, cycles per tensor-core instruction of that width, epilogue, bytes) and the cheapest is
   * kept. eval_variant, when set, replaces eval: it is called once per variant of a node (variant 0 for nodes that
   * have none), the minimum becomes the node's cost and the arg-min is recorded for the step. */
  fluid_eval_variant_fn eval_variant;
  /* Per graph op (the LINEAR / BMM op a GEMM step is built on): a variant code to run that step with instead of the
   * rated best; 0 or an entry beyond n_op_variant leaves the choice to the planner; a code the step's shape cannot
   * take is ignored. Copied by fluid_plan. */
  const int32_t* op_variant;
  int32_t n_op_variant;
  int32_t no_inplace;       /* 0 (default): a rotary-embedding, element-wise or residual-epilogue step whose input dies
                               with it writes its result over that input (one arena record, union lifetime);
                               1: every result gets a slice of its own */
  int32_t redzone_bytes;    /* debugging aid (0 = none): every activation slice is followed by this many bytes (rounded up
                               to 256) that no kernel may write. In a no_reuse plan the slices are disjoint, so a caller
                               that fills the arena with a pattern before fluid_run can check the zones afterwards: an
                               out-of-bounds store of any kernel shows up without a memory checker */
  int32_t no_norm_split;    /* 0 (default): an RMS normalisation that sits between a residual GEMM step and GEMM steps that
                               all run as CTA pairs is split across them (the first also writes bf16(x * gain) and per-slab
                               sums of squares, the others scale their rows by 1 / rms): no launch of its own, and the
                               normalised tensor is never stored; 1: it stays a step */
} fluid_plan_options;

typedef enum {
  FLUID_K_EMBED = 0, FLUID_K_NORM = 1, FLUID_K_GEMM_SIMT = 2, FLUID_K_GEMM_TC = 3,
  FLUID_K_SOFTMAX = 4, FLUID_K_ROPE = 5, FLUID_K_ELTWISE = 6, FLUID_K_PERMUTE = 7,
  FLUID_K_SELECT_LAST = 8, FLUID_K_ATTN = 9, FLUID_K_ATTN_DECODE = 10, FLUID_K_GEMM_ROWS = 11, FLUID_K_COUNT = 12
} fluid_kernel_id;

typedef struct fluid_step_info {
  int32_t kernel;        /* fluid_kernel_id */
  int32_t variant;       /* kernel-specific (GEMM: the implementation variant that runs, as chosen by the planner's
                            rating or the caller's eval_variant / op_variant: bit0 A MN-major, bit1 B MN-major, bits 8-19 tile N,
                            bits 20-23 grouped siblings, bits 24-27 split-K factor, bit 28: the split
                            runs as one thread-block cluster per output tile, bit 29: pairs of CTAs share
                            256 x 256 tiles, bit 30: the rotary embedding of the first projections of the group runs in the epilogue. GEMM_ROWS: bits 20-23 grouped siblings, bit 29: SiLU(gate) * up is
                            applied in the launch, bit 30: the preceding RMS normalisation runs in the launch.
                            ATTN_DECODE: bits 0-7 head dim, bits 8-15 query heads per key/value head, bit 16:
                            the rotary embedding of query and key runs in the launch) */
  int32_t n_ops;         /* graph ops folded into this step */
  int32_t ops[8];
  int32_t n_in, n_out;   /* tensors read / written (graph tensor ids) */
  int32_t in_ids[8];
  int32_t out_ids[4];
  double cost;           /* modelled (or user-evaluated) time, seconds */
  double flops;          /* algorithmic floating-point operations */
  double bytes;          /* algorithmic bytes moved to and from device memory */
} fluid_step_info;

/* ---- graph construction (host) --------------------------------------------------------- */
FLUID_API int fluid_graph_create(fluid_graph_t** g);
FLUID_API void fluid_graph_destroy(fluid_graph_t* g);
/* dims: rank ints, logical shape. Returns the tensor id in *tensor_id (ids count from 0). */
FLUID_API int fluid_graph_add_tensor(fluid_graph_t* g, int dtype, int rank, const int64_t* dims, int kind,
                           int* tensor_id);
/* Shapes and dtypes are checked against the operator's definition; attrs may be NULL. */
FLUID_API int fluid_graph_add_op(fluid_graph_t* g, int op_kind, int n_in, const int* in_ids, int n_out,
                       const int* out_ids, const fluid_op_attrs* attrs, int* op_id);

/* ---- planning (host only; touches no device) --------------------------------------------
 * Linearises the graph, splits it into sequences (Algorithms 1-2), runs the per-sequence
 * dynamic programme over layouts (Eq. 1, Algorithm 3), merges by majority vote, lowers to a
 * list of kernel steps, computes lifetimes and places every activation with Greedy-by-Size
 * (Algorithm 4). cands or opts may be NULL (canonical only / defaults). */
FLUID_API int fluid_plan(const fluid_graph_t* g, const fluid_layout_candidates* cands,
                      const fluid_plan_options* opts, fluid_plan_t** plan);
FLUID_API void fluid_plan_destroy(fluid_plan_t* plan);
FLUID_API void fluid_plan_default_options(fluid_plan_options* opts);

/* The implementation variants the GEMM step built on graph op `op_id` can run with under the plan's layouts
 * (codes as in fluid_plan_options), and the one the plan runs (*chosen). codes may be NULL to query the count.
 * An op that is not the anchor of a tensor-core GEMM step has no variants (*n = 0, *chosen = 0). */
FLUID_API int fluid_plan_gemm_variants(const fluid_plan_t* plan, int op_id, int* codes, int capacity, int* n, int* chosen);

/* Peak bytes of the arena, header included; the caller allocates exactly this much. */
FLUID_API size_t fluid_plan_arena_bytes(const fluid_plan_t* plan);
/* Sum of all slices without reuse, and the largest simultaneously-live sum (both + header). */
FLUID_API size_t fluid_plan_arena_naive_bytes(const fluid_plan_t* plan);
FLUID_API size_t fluid_plan_arena_live_bound_bytes(const fluid_plan_t* plan);
/* Total modelled cost of the chosen layouts and of the all-canonical assignment, seconds. */
FLUID_API double fluid_plan_cost(const fluid_plan_t* plan);
FLUID_API double fluid_plan_canonical_cost(const fluid_plan_t* plan);

/* Per tensor: chosen layout index and permutation (rank ints); offset/bytes of its arena slice
 * (offset -1 when it is not arena-resident: input, output, constant, or folded away by fusion);
 * inclusive step lifetime; alias_of = the tensor whose storage it shares (itself if none).
 * Any out pointer may be NULL. */
FLUID_API int fluid_plan_tensor_info(const fluid_plan_t* plan, int tensor_id, int* layout_index, int* perm,
                           int64_t* offset, int64_t* bytes, int* first_step, int* last_step,
                           int* alias_of);
/* Arena slices. A tensor held in fp32 with a bf16 twin owns two slices; a GEMM step that splits its
 * k range across CTAs owns a scratch slice alive during that step only (tensor_id -1). record_id is
 * unique (tensor id; tensor id + number of tensors for a twin; 2 * number of tensors + step for
 * scratch); storage_dtype is the fluid_dtype the slice holds. Any out pointer may be NULL. */
FLUID_API int fluid_plan_num_records(const fluid_plan_t* plan);
FLUID_API int fluid_plan_record_info(const fluid_plan_t* plan, int index, int* record_id, int* tensor_id,
                           int* is_twin, int* storage_dtype, int64_t* offset, int64_t* bytes,
                           int* first_step, int* last_step);
FLUID_API int fluid_plan_num_steps(const fluid_plan_t* plan);
FLUID_API int fluid_plan_step_info(const fluid_plan_t* plan, int step, fluid_step_info* info);
/* The sequences of Algorithm 2, as node ids (= op ids when fusion is 0). */
FLUID_API int fluid_plan_num_sequences(const fluid_plan_t* plan);
FLUID_API int fluid_plan_sequence(const fluid_plan_t* plan, int index, int* node_ids, int capacity, int* length);

/* ---- constants (weights live outside the arena; the paper keeps them in read-only data) ----
 * bind: dev_ptr must already hold the tensor in the plan's layout for it and stay valid.
 * pack: one-time device-side re-layout of a canonical constant into the planned layout. */
FLUID_API int fluid_plan_bind_constant(fluid_plan_t* plan, int tensor_id, const void* dev_ptr);
FLUID_API int fluid_pack_constant(const fluid_plan_t* plan, int tensor_id, const void* dev_src_canonical,
                        void* dev_dst, fluid_stream stream);

/* ---- execution -----------------------------------------------------------------------------
 * Launches every step of the plan on `stream` and returns without synchronising. arena_ptr:
 * device, FLUID_ARENA_ALIGN-aligned, fluid_plan_arena_bytes() long. inputs/outputs: host arrays
 * of device pointers in declaration order, each 16-byte aligned. No device memory is allocated,
 * freed or copied to the host. Launch errors are reported as FLUID_ECUDA. Runs of one plan that
 * share an arena must not overlap in time. */
FLUID_API int fluid_run(fluid_plan_t* plan, void* arena_ptr, const void* const* inputs, void* const* outputs,
              fluid_stream stream);
/* As fluid_run, but brackets each step with CUDA events and, after synchronising the stream,
 * writes per-step milliseconds to step_ms[fluid_plan_num_steps()]. For measurement only. */
FLUID_API int fluid_run_profiled(fluid_plan_t* plan, void* arena_ptr, const void* const* inputs,
                       void* const* outputs, fluid_stream stream, float* step_ms);
/* Synchronises `stream`, reads the arena header and reports in *device_status 0 or the code a
 * kernel left: when one of its bounded waits expired (returns FLUID_ETIMEOUT), or, bit 0x10, when a
 * CACHED_ATTENTION step read a position outside its cache (returns FLUID_EINVAL). */
FLUID_API int fluid_status(const fluid_plan_t* plan, const void* arena_ptr, fluid_stream stream,
                 int* device_status);

/* ---- one GEMM that allocates nothing (the paper has no counterpart) ---------------------------
 * C[m,n] = A[m,k] . B[n,k]^T (+ bias[n]), all bf16 device buffers the caller owns (A and B with k
 * contiguous, C with n contiguous, 16-byte aligned; bias may be NULL), fp32 accumulate, run by the
 * same tensor-core kernel as the planned GEMM steps in its split-K form.
 *
 * Who it is for: callers that want this one product outside any plan and cannot obtain device memory
 * for it. Every other route through this library makes the caller allocate an arena first
 * (fluid_plan_arena_bytes); a host thread in the middle of a latency-critical serving loop, a plugin
 * whose host framework owns the allocator, or a process whose memory budget was fixed at start-up has
 * no such allocation to give, and cudaMalloc there would stall the device or break the host's
 * accounting. This call therefore takes nothing but inputs and outputs: the split-K partial tiles and
 * arrival counters live in one fixed array inside the library's device image (8 MiB + 256 bytes, held
 * by every GPU that loads the library until the process exits). It calls no cudaMalloc / cudaFree and
 * no allocating library routine.
 *
 * Limits and rules:
 *  - k and n multiples of 8; the split-K scratch the shape needs (n_tiles * split * 128 * tile_n * 4
 *    bytes; 0 for shapes large enough to need no split) must fit the 8 MiB array, otherwise
 *    FLUID_EINVAL with a message naming both figures.
 *  - The first call on each device looks up the array's device address (with that device current);
 *    make that first call before any stream capture begins.
 *  - All calls share the one array: it is re-zeroed where needed at the start of every call, and two
 *    calls whose kernels overlap on the GPU (different streams, or graphs replayed concurrently) race.
 *  - Asynchronous on `stream`; launch errors come back as FLUID_ECUDA. A bounded wait that expires
 *    inside the kernel is NOT reported by this call: the kernel records a code in the array's first
 *    word, drains and returns, leaving C partly unwritten. fluid_static_scratch_status reads it. */
FLUID_API int fluid_gemm_bf16_static_scratch(const void* dev_a, const void* dev_b, const void* dev_bias, void* dev_c,
                                   int m, int n, int k, fluid_stream stream);
/* Status of the last fluid_gemm_bf16_static_scratch call on the current device (the paper has no
 * counterpart). Synchronises `stream`, then copies the status word out of the static array with one
 * 4-byte cudaMemcpy (no allocation). *device_status = 0 and FLUID_OK when every wait completed (or
 * when no call has been made on this device yet); a non-zero code and FLUID_ETIMEOUT when a bounded
 * wait gave up, in which case C is incomplete and the array's arrival counters are stale (the next
 * call re-zeroes them). Like fluid_status, it must not overlap a later call on another stream. */
FLUID_API int fluid_static_scratch_status(fluid_stream stream, int* device_status);

FLUID_API const char* fluid_last_error(void);
/* Number of kernel launches issued by this library in this process (for launch accounting). */
FLUID_API int64_t fluid_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FLUID_H */
