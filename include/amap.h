/*
 * amap.h -- composed affine copies: C ABI.
 *
 * A chain of layout operators (reshape, transpose, strided slice, concat, pad,
 * im2col-style window gather, ...) is a sequence of loop nests, each holding
 * one element-wise load  v = t_l[C_l i + b_l]  feeding one store
 * t_s[C_s i + b_s] = v  (the paper's Section 2, equations (load) and (store),
 * and the pair pattern of Section 2.1).  amap_compose() removes every
 * intermediate tensor by composing the access maps on the host (Section 2.1,
 * equations (1) and (2), repeated until no pair is left); amap_plan() chooses
 * a CUDA kernel family for what remains; amap_execute() runs the single
 * remaining copy on a caller-supplied stream.
 *
 * Conventions
 *  - Tensors are dense, row-major; elements are opaque patterns of elem_size
 *    bytes (1, 2, 4, 8 or 16).  No floating-point arithmetic happens anywhere.
 *  - Every function returns AMAP_OK (0) or a negative amap_status.  Out-handles
 *    are written only on success.  Nothing throws, exits or prints (unless the
 *    environment variable AMAP_LOG is set to something other than 0, which
 *    prints composed pieces and the reason of a failure to stderr).
 *  - Host arrays passed in are read during the call and copied; the caller
 *    keeps ownership.  Handles returned are owned by the library until the
 *    matching *_destroy call.  Device buffers are always the caller's.
 *  - "host" / "device" is stated for every pointer argument.
 */
#ifndef AMAP_H_
#define AMAP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum amap_status {
  AMAP_OK = 0,
  AMAP_EINVAL = -1,               /* null pointer, bad rank / bounds / ids / elem_size             */
  AMAP_ESTORE_NOT_INJECTIVE = -2, /* a store map writes one element twice: it has no reverse       */
  AMAP_EOOB = -3,                 /* an unguarded access can leave its tensor                      */
  AMAP_EUNDEFINED = -4,           /* an element that is read (or an output element) is never written*/
  AMAP_EOVERLAP = -5,             /* two statements write the same element                         */
  AMAP_EOVERFLOW = -6,            /* an offset or element count does not fit the integer width used*/
  AMAP_EALIGN = -7,               /* a device pointer is less aligned than the plan requires       */
  AMAP_ECUDA = -8,                /* a CUDA runtime call failed; see amap_last_cuda_error()        */
  AMAP_EUNSUPPORTED = -9,         /* valid input the host algebra cannot compose affinely          */
  AMAP_ENOMEM = -10,
  AMAP_ETOOLARGE = -11            /* the plan does not fit the fixed table of amap_execute_static   */
} amap_status;

#define AMAP_CONST (-1) /* amap_access.tensor of a load that yields the statement's fill_bits */
#define AMAP_MAX_LOOPS 12
#define AMAP_MAX_RANK 8

/* One access t[C i + b] (Section 2, equations (load)/(store)).  host pointers. */
typedef struct amap_access {
  int32_t tensor;   /* id of the tensor accessed, or AMAP_CONST (loads only)       */
  int32_t rank;     /* m, the tensor's rank; 1 for a tensor of higher rank = its flat row-major view */
  const int64_t *C; /* m x n_loops, row-major                                       */
  const int64_t *b; /* m                                                            */
} amap_access;

/* One loop nest = one load/store pair (Section 2.1).  For every i in the box
 * 0 <= i_j < bounds[j]:  store.tensor[C_s i + b_s] = load.tensor[C_l i + b_l]. */
typedef struct amap_stmt {
  int32_t n_loops;       /* n, 0..AMAP_MAX_LOOPS                                    */
  const int64_t *bounds; /* n extents, each >= 0 (host)                             */
  amap_access load;
  amap_access store;
  int32_t guarded;    /* 1: a load index outside load.tensor's shape yields fill_bits instead of being an error */
  uint64_t fill_bits; /* low elem_size bytes (elements wider than 8 bytes: zero-extended) */
} amap_stmt;

typedef struct amap_tensor {
  int32_t rank;         /* 1..AMAP_MAX_RANK                                          */
  const int64_t *shape; /* rank extents (host)                                       */
} amap_tensor;

/* A whole chain: external inputs, intermediates and one output tensor; the
 * statements in an order in which every tensor is written before it is read. */
typedef struct amap_chain {
  int32_t n_tensors;
  const amap_tensor *tensors;
  int32_t n_stmts;
  const amap_stmt *stmts;
  int32_t n_inputs;
  const int32_t *inputs; /* tensor ids bound to device pointers at execute time, in this order */
  int32_t output;        /* tensor id of the result                                            */
  int32_t elem_size;     /* 1, 2, 4, 8 or 16 bytes                                             */
} amap_chain;

typedef struct amap_builder amap_builder;
typedef struct amap_map amap_map;
typedef struct amap_plan_t amap_plan_t;

/* ---------------------------------------------------------------------------
 * Chain builder: emits the statements of the common operators in the paper's
 * form (Section 2.1 names the families).  Each call appends one tensor and the
 * statement(s) that define it and returns the new tensor's id in *out.
 * All array arguments are host pointers with `rank` entries unless stated.
 * ------------------------------------------------------------------------- */
int amap_builder_create(int32_t elem_size, amap_builder **out);
void amap_builder_destroy(amap_builder *b);
/* an external input of the given shape */
int amap_builder_input(amap_builder *b, int32_t rank, const int64_t *shape, int32_t *out);
/* same flat order, new shape (element counts must agree) */
int amap_builder_reshape(amap_builder *b, int32_t src, int32_t rank, const int64_t *shape, int32_t *out);
/* out.shape[d] = in.shape[perm[d]] */
int amap_builder_transpose(amap_builder *b, int32_t src, int32_t rank, const int32_t *perm, int32_t *out);
/* out[o] = in[start + step*o], step >= 1, 0 <= start <= stop <= in.shape */
int amap_builder_slice(amap_builder *b, int32_t src, int32_t rank, const int64_t *start, const int64_t *stop,
                       const int64_t *step, int32_t *out);
/* join n tensors (ids in srcs) on `axis` */
int amap_builder_concat(amap_builder *b, int32_t n, const int32_t *srcs, int32_t axis, int32_t *out);
/* lo/hi elements of fill_bits before/after every axis (one guarded statement) */
int amap_builder_pad(amap_builder *b, int32_t src, int32_t rank, const int64_t *lo, const int64_t *hi,
                     uint64_t fill_bits, int32_t *out);
/* NHWC [N,H,W,C] -> [N*Ho*Wo, kh*kw*C] with column (r*kw+s)*C+c reading
 * in[n, ho*stride+r-pad, wo*stride+s-pad, c], zero outside (one guarded, non-injective load) */
int amap_builder_window(amap_builder *b, int32_t src, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                        int32_t *out);
/* The same gather with taps `dilation` pixels apart and a choice of column order: tap (r, s) of output pixel
 * (ho, wo) reads in[n, ho*stride + r*dilation - pad, wo*stride + s*dilation - pad, c], zero outside;
 * Ho = (H + 2*pad - dilation*(kh-1) - 1)/stride + 1, likewise Wo.  AMAP_WINDOW_COLS_RSC: column (r*kw+s)*C+c
 * (channel fastest, as amap_builder_window); AMAP_WINDOW_COLS_CRS: column (c*kh+r)*kw+s (tap fastest, the order
 * of NCHW im2col).  Still one guarded load/store pair in the paper's form (Section 2.1). */
#define AMAP_WINDOW_COLS_RSC 0
#define AMAP_WINDOW_COLS_CRS 1
int amap_builder_window_ex(amap_builder *b, int32_t src, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                           int32_t dilation, int32_t column_order, int32_t *out);
/* broadcast: out[o] = in[o mod in.shape] with out.shape[d] = reps[d]*in.shape[d] (the paper's repeat/tile family) */
int amap_builder_tile(amap_builder *b, int32_t src, int32_t rank, const int64_t *reps, int32_t *out);
/* every element `count` times in a row along `axis`: out[.., i*count + j, ..] = in[.., i, ..] (a load that ignores
 * one loop; Section 2.1 names repeat among the operators whose copies are eliminated) */
int amap_builder_repeat(amap_builder *b, int32_t src, int32_t axis, int64_t count, int32_t *out);
/* cut `src` along `axis` into n_parts consecutive tensors of the given sizes (they must add up to the extent;
 * Section 2.1 names split); outs receives n_parts tensor ids (host array, caller-owned).  Each part is a tensor
 * of its own: compose once per part that is wanted as an output. */
int amap_builder_split(amap_builder *b, int32_t src, int32_t axis, int32_t n_parts, const int64_t *sizes,
                       int32_t *outs);
/* A tensor computed by an operator that is NOT a layout operator (a convolution, a matmul, ...) from the tensors
 * `ins` (host array of n_ins ids).  Data-movement elimination stops at such an operator (Section 2.1 eliminates
 * load/store PAIRS; the paper's evaluation, Section 3, keeps what feeds compute): the new tensor is bound at execute
 * time like an external input (its position in amap_chain.inputs follows the inputs declared before it), the
 * statements behind it compose into reads of it, and the statements before it compose into the tensors in `ins`,
 * which the caller asks for as outputs of a map of their own (amap_compose_multi) and hands to the operator. */
int amap_builder_opaque(amap_builder *b, int32_t n_ins, const int32_t *ins, int32_t rank, const int64_t *shape,
                        int32_t *out);
/* declare a tensor that raw statements will define */
int amap_builder_tensor(amap_builder *b, int32_t rank, const int64_t *shape, int32_t *out);
/* append one raw statement (deep-copied) */
int amap_builder_stmt(amap_builder *b, const amap_stmt *stmt);
/* a view of everything built so far with `output` as the result; valid until the next builder call */
int amap_builder_chain(amap_builder *b, int32_t output, const amap_chain **out);

/* ---------------------------------------------------------------------------
 * amap_compose: Section 2.1, equations (1) and (2), to the fixpoint.
 * Host only, no CUDA.  The result is a list of PIECES, each one loop nest in
 * the paper's form over the FLAT (rank-1, row-major) views of an external
 * input and of the output:
 *     out.flat[C_s i + b_s] = in[input].flat[C_l i + b_l]      for i in the box,
 * so C_l and C_s are 1 x n_loops (element strides) and b_l, b_s scalars.
 * Pieces write pairwise disjoint sets that together cover the output.
 * Errors: EINVAL, ESTORE_NOT_INJECTIVE, EOOB, EUNDEFINED, EOVERLAP,
 * EOVERFLOW, EUNSUPPORTED (e.g. a reshape whose factors do not line up with
 * the loops that read it), ENOMEM.
 * ------------------------------------------------------------------------- */
int amap_compose(const amap_chain *chain, amap_map **out_map);
/* amap_compose with options.  AMAP_COMPOSE_NO_FUSE keeps EVERY intermediate tensor as a temporary, i.e. runs the
 * chain operator by operator as the paper's Section 2.1 finds it before the optimisation (the comparison baseline). */
#define AMAP_COMPOSE_NO_FUSE 1u
/* Quasi-affine pieces.  Where a pair has no affine composition (a reshape whose factors do not line up with the loops
 * around it: the reverse of the store needs floor-division and remainder, which the paper leaves to ISL, Section
 * 2.1), amap_compose can still eliminate the intermediate with a piece whose source offset is
 *     b_l + sum_k digit_stride[k] * digit_k(f0 + F i),
 * digit_k being the digits of the affine form f0 + F i in the mixed radix digit_radix[] (innermost last).  By default
 * it does so only where a contiguous run of at least 16 bytes survives on both sides (one division chain per run);
 * otherwise the intermediate stays a temporary (two passes of vector kernels beat one pass of scattered element
 * accesses).  AMAP_COMPOSE_QUASI_AFFINE: wherever a pair allows one, also in place of an affine composition (for
 * measurements and tests); AMAP_COMPOSE_NO_QUASI_AFFINE: never. */
#define AMAP_COMPOSE_QUASI_AFFINE 2u
#define AMAP_COMPOSE_NO_QUASI_AFFINE 4u
int amap_compose_ex(const amap_chain *chain, uint32_t flags, amap_map **out_map);
/* Several results from one chain (Section 2.1 names split; its last paragraph repeats the elimination until no pair
 * is left, over the whole graph): `outputs` (host array of n_outputs distinct tensor ids, 1..8; chain->output is
 * ignored) are all composed back to the external inputs in ONE map.  Their pieces form the map's last stage side by
 * side (amap_piece.output says which output a piece writes), so one amap_execute_multi launch writes all of them --
 * the parts of a split cost one launch instead of one per part.  A tensor may be an output and be read by later
 * statements as well. */
int amap_compose_multi(const amap_chain *chain, int32_t n_outputs, const int32_t *outputs, uint32_t flags,
                       amap_map **out_map);
int amap_map_num_outputs(const amap_map *map, int32_t *n);
/* elements of output k (amap_map_sizes reports output 0) */
int amap_map_output_numel(const amap_map *map, int32_t k, int64_t *numel);
void amap_map_destroy(amap_map *map);

/* Stages.  A map normally has ONE stage: all intermediates are gone.  Where a load/store pair cannot be
 * eliminated affinely (Section 3 of the paper reports such a leftover pair too: 123 of 124), the intermediate
 * stays as a TEMPORARY: an earlier stage writes it and later stages read it.  Stage s owns pieces
 * [first_piece, first_piece + n_pieces) of the piece list and writes temporary *dst_temp (0-based) or, when
 * *dst_temp is -1, the output(s) -- the last stage, whose pieces name their output in amap_piece.output; an
 * amap_piece.input >= n_inputs names temporary (input - n_inputs).
 * Temporaries live in device memory that amap_plan allocates. */
int amap_map_num_stages(const amap_map *map, int32_t *n);
int amap_map_get_stage(const amap_map *map, int32_t s, int32_t *first_piece, int32_t *n_pieces, int32_t *dst_temp,
                       int64_t *dst_numel);

/* a constraint  0 <= offset + sum_k coef[k] * i_k < extent  on the loop indices */
typedef struct amap_constraint {
  const int64_t *coef; /* n_loops (host, owned by the map) */
  int64_t offset;
  int64_t extent;
} amap_constraint;

/* One piece of a composed map: a loop nest in the paper's form (Section 2, equations (load)/(store)) after
 * Section 2.1's rewrite, i.e. the reader's store with the load g' = f_l o f_s' o f_l' of equation (2) put in its
 * place.  It differs from amap_stmt only in that both tensors are addressed through their flat views (rank 1,
 * so C_l and C_s are single rows and b_l, b_s scalars) and that guards / domain constraints are spelled out. */
typedef struct amap_piece {
  int32_t n_loops;
  const int64_t *bounds; /* n_loops (host, owned by the map)                                   */
  int32_t input;         /* position in amap_chain.inputs of the tensor read, or AMAP_CONST    */
  const int64_t *C_l;    /* n_loops source strides in elements (NULL for AMAP_CONST)           */
  int64_t b_l;
  const int64_t *C_s; /* n_loops destination strides in elements                               */
  int64_t b_s;
  int32_t n_guards; /* where any guard fails the piece stores fill_bits instead of loading     */
  const amap_constraint *guards;
  int32_t n_domain; /* where any of these fails the loop point is not part of the piece        */
  const amap_constraint *domain;
  uint64_t fill_bits;
  int32_t output; /* which output of the map the piece writes (0 unless amap_compose_multi named several) */
  /* quasi-affine pieces only (n_digits > 0; C_l is all zero then): see AMAP_COMPOSE_QUASI_AFFINE */
  int32_t n_digits;
  const int64_t *digit_radix;  /* n_digits (host, owned by the map) */
  const int64_t *digit_stride; /* n_digits source strides in elements */
  const int64_t *F;            /* n_loops coefficients of the inner affine form */
  int64_t f0;
} amap_piece;

/* number of pieces of the composed map (all stages): the load/store pairs that are left once Section 2.1's
 * elimination has reached its fixpoint */
int amap_map_num_pieces(const amap_map *map, int32_t *n);
/* piece k in the form above (Section 2.1, equation (2): the rewritten reader); *out receives views into the
 * map, valid until amap_map_destroy.  host pointers. */
int amap_map_get_piece(const amap_map *map, int32_t k, amap_piece *out);
/* element counts of the external inputs (n_inputs entries written to in_numel, a host array of the caller) and of
 * the output: the tensors t_l and t_s of Section 2 that survive the elimination and must exist in device memory */
int amap_map_sizes(const amap_map *map, int32_t *n_inputs, int64_t *in_numel /* may be NULL */, int64_t *out_numel,
                   int32_t *elem_size);

/* ---------------------------------------------------------------------------
 * amap_plan: choose a kernel family per piece and build the launch table.
 * (Section 2.2 of the paper: the memory references that remain after the
 * elimination are compulsory, and the way they are laid out and issued must
 * let them use the available memory bandwidth in full.  There that is a
 * mapping of tensors to scratchpad banks; here it is the choice of access
 * width, tile shape and loop order per piece.)
 * `device` is a CUDA ordinal: the call makes it current, uploads a small
 * descriptor table to device memory owned by the plan, and restores the
 * previous device.  device = -1 gives a dry plan (no CUDA call at all) whose
 * statistics and kernel choices can be read but which amap_execute refuses
 * with AMAP_EINVAL.  Before anything is uploaded the planner walks the table
 * on the host with the kernel's own index arithmetic and checks that every
 * address stays inside its buffer and is aligned to the access width; a
 * violation gives AMAP_EOVERFLOW.  A plan is immutable and may be executed
 * any number of times, on any stream of its device, concurrently.
 * ------------------------------------------------------------------------- */
typedef enum amap_kernel_kind {
  AMAP_KERNEL_AUTO = 0,
  AMAP_KERNEL_GATHER = 1,    /* one element per thread, full index arithmetic, guards; handles every piece */
  AMAP_KERNEL_COPY = 2,      /* innermost loop contiguous on both sides: 16-byte vector runs               */
  AMAP_KERNEL_TRANSPOSE = 3, /* the fastest source loop differs from the fastest destination loop: smem tile */
  AMAP_KERNEL_FILL = 4       /* no source: vector stores of the constant                                   */
} amap_kernel_kind;

/* amap_plan_opts.flags: launch the kernels without programmatic dependent launch (by default a kernel's
 * prologue may overlap the tail of the kernel before it on the stream; it touches no buffer until that one is done) */
#define AMAP_PLAN_NO_PDL 1
/* do not prefetch a block's first source lines into L2 while the previous kernel on the stream drains */
#define AMAP_PLAN_NO_PREFETCH 2
/* (The environment variable AMAP_PREFETCH_DISTANCE, read by amap_plan, overrides how many blocks ahead the
 * transpose kernel prefetches; the default is the number of blocks resident on the device at once.) */

typedef struct amap_plan_opts {
  int32_t force_kernel;     /* amap_kernel_kind; AUTO picks per piece; a family that cannot run a piece falls back to GATHER */
  int32_t pointer_align;    /* bytes every src/dst base pointer is promised to be aligned to (0 = elem_size; 16 enables vectors) */
  int32_t flags;            /* AMAP_PLAN_* bits */
  int32_t reserved[5];      /* must be zero */
} amap_plan_opts;

typedef struct amap_stats {
  int64_t bytes_read;    /* unique source bytes the composed copy must read   */
  int64_t bytes_written; /* output bytes written (copied + filled)            */
  int64_t bytes_filled;  /* the part of bytes_written that has no source      */
  int32_t n_pieces;
  int32_t n_launches;     /* kernels one amap_execute enqueues                 */
  int32_t kernel_kind[4]; /* pieces planned per family: [0] gather [1] copy [2] transpose [3] fill */
  int32_t n_stages;       /* 1 unless the map keeps temporaries */
  int32_t n_descriptors;  /* launch descriptors behind the pieces (a piece may be cut into several)   */
} amap_stats;

int amap_plan(const amap_map *map, int device, const amap_plan_opts *opts /* host, may be NULL */,
              amap_plan_t **out_plan);
void amap_plan_destroy(amap_plan_t *plan);
/* the compulsory traffic of the plan (Section 2.2: what cannot be eliminated): each unique source byte once,
 * each output byte once; also how many kernels an execute enqueues and the family chosen per piece */
int amap_plan_stats(const amap_plan_t *plan, amap_stats *out /* host */);
/* kernel family chosen for piece k (an amap_kernel_kind) */
int amap_plan_piece_kernel(const amap_plan_t *plan, int32_t k, int32_t *kind);

/* Launch k of the plan (0 <= k < amap_stats.n_launches), in the order amap_execute enqueues them: which kernel
 * runs, over how many descriptors and blocks.  For inspection and tests; AMAP_EINVAL for a k out of range. */
enum {
  AMAP_LAUNCH_AFFINE = 0,            /* per-unit copy / gather                                         */
  AMAP_LAUNCH_STRIP = 1,             /* strips of units along one loop                                 */
  AMAP_LAUNCH_TRANSPOSE = 2,         /* tiled transpose, `access` bytes (16, 8, 4, 2) per global access */
  AMAP_LAUNCH_TRANSPOSE_SHIFTED = 3, /* tiled transpose onto destination rows that are not 16-byte aligned */
  AMAP_LAUNCH_TRANSPOSE_REALIGN = 4, /* tiled transpose from source rows that are not 16-byte aligned  */
  AMAP_LAUNCH_TRANSPOSE_FLAT = 5,    /* transpose by panels that are contiguous in the destination     */
  AMAP_LAUNCH_TRANSPOSE_FLAT_SOURCE = 6 /* transpose by panels that are contiguous in the source       */
};
typedef struct amap_launch_info {
  int32_t kernel;        /* AMAP_LAUNCH_*                                               */
  int32_t access;        /* bytes per global access (affine / strip: the unit width)    */
  int32_t n_descriptors; /* descriptors the launch covers                               */
  int32_t stage;         /* stage of the map the launch belongs to                      */
  uint32_t n_blocks;
  int32_t threads;       /* threads per block                                           */
  int32_t smem_bytes;    /* dynamic shared memory per block (0: the kernel's static tile) */
  int32_t wide_offsets;  /* 1: 64-bit byte offsets                                      */
} amap_launch_info;
int amap_plan_launch_info(const amap_plan_t *plan, int32_t k, amap_launch_info *out /* host */);

/* ---------------------------------------------------------------------------
 * amap_execute: the surviving copy (the data movement Section 2.1 cannot
 * remove and Section 2.2 wants run at full memory bandwidth).
 *   src_dev_ptrs  host array of n_inputs DEVICE pointers, in amap_chain.inputs order (the entry of an input
 *                 that no piece of the map reads may be NULL)
 *   dst_dev_ptr   DEVICE pointer to the output (out_numel * elem_size bytes)
 *   cuda_stream   a cudaStream_t (NULL = the legacy default stream)
 * Enqueues the plan's kernel(s) -- one per kernel family present in the map,
 * one in all for each of the common operator chains -- and returns without
 * synchronising or allocating.  Source and destination must not overlap (AMAP_EINVAL if the
 * byte ranges do).  Pointers must be
 * aligned to the plan's pointer_align, else AMAP_EALIGN and nothing is
 * enqueued.  Launch failures give AMAP_ECUDA.
 * ------------------------------------------------------------------------- */
int amap_execute(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *dst_dev_ptr, void *cuda_stream);
/* The same for a map with several outputs (amap_compose_multi): dst_dev_ptrs is a host array of n_outputs DEVICE
 * pointers in the order the outputs were named.  No buffer may overlap another (sources with destinations,
 * destinations with each other): AMAP_EINVAL.  amap_execute, amap_execute_host and amap_execute_static take plans
 * of single-output maps only (AMAP_EINVAL otherwise). */
int amap_execute_multi(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *const *dst_dev_ptrs,
                       void *cuda_stream);

/* Same copy with HOST buffers: uploads the inputs, runs the plan, downloads
 * the output and waits.  Uses device staging memory owned by the plan
 * (allocated on first use).  src_host_ptrs: host array of n_inputs HOST
 * pointers; dst_host_ptr: HOST.  Pinned host memory makes the copies faster
 * but is not required.  When the outermost loop of the whole map is a batch
 * loop (slab k of the output needs only slab k of every input) the call works
 * slab by slab on two more streams of its own, so that upload, kernel and
 * download overlap; the result is the same.  The staging memory and the extra
 * streams belong to the plan: calls on ONE plan must not run at the same time
 * (amap_execute on the same plan is unaffected). */
int amap_execute_host(amap_plan_t *plan, const void *const *src_host_ptrs, void *dst_host_ptr, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * amap_execute_static: amap_execute for callers that are not allowed to
 * allocate device memory.  (The paper has no counterpart; this is a service of
 * the library.)  Typical callers: a plug-in running inside a framework that
 * owns all device memory, a real-time or serving loop in which cudaMalloc's
 * implicit device-wide synchronisation is not acceptable, code that runs after
 * the memory budget has been handed out.  Such a caller makes a DRY plan
 * (amap_plan with device = -1, which touches no CUDA API) and passes it here;
 * a plan made for the current device is accepted too.
 *
 * Instead of the plan's own table in cudaMalloc'ed memory, the kernels read
 * their descriptors from a fixed array that is part of the library image
 * (64 descriptors, about 70 KB; every GPU on which the library is loaded
 * holds it until the process exits).  The call enqueues, on `cuda_stream`,
 * small kernels that carry the plan's descriptors in their parameters and
 * write them into that array, and behind them the same kernels as
 * amap_execute.  It calls no cudaMalloc / cudaFree, no allocating library
 * routine and no host-to-device copy, and waits for nothing: neither the host
 * nor the stream is synchronised.
 *
 *  - Runs on the CURRENT device; src/dst pointers and the stream must belong
 *    to it.  Arguments, alignment rules and refusals (null pointers, AMAP_EALIGN,
 *    AMAP_EINVAL for source and destination byte ranges that overlap) are those
 *    of amap_execute.  A plan made for another device gives AMAP_EINVAL.
 *  - A plan with more than 64 descriptors is refused with AMAP_ETOOLARGE and
 *    nothing is enqueued (compose fewer operators per call, or use amap_execute).
 *    A plan whose map keeps temporaries (more than one stage) is refused with
 *    AMAP_EUNSUPPORTED: temporaries need device memory.
 *  - The first call on each device looks up the array's device address
 *    (cudaGetSymbolAddress) and the device's multiprocessor count and keeps
 *    both for later calls; make that first call before starting any stream
 *    capture on that device.  cudaDeviceReset invalidates what was kept: do not
 *    call this function again in a process that has reset the device.
 *  - All calls on one device share the one array, which still holds the
 *    previous call's descriptors until the next call's upload kernels overwrite
 *    them.  Calls are safe back to back on ONE stream, issued by one host thread
 *    at a time (two threads enqueueing on the same stream could interleave their
 *    uploads and copies).  Two calls that can overlap on the GPU (different
 *    streams without an ordering between them) race on the array: order them
 *    with events or use amap_execute for one of them.
 *  - A dry plan assumes a 148-multiprocessor device for its L2 look-ahead
 *    distances; this call rescales them to the device it runs on.
 * ------------------------------------------------------------------------- */
int amap_execute_static(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *dst_dev_ptr, void *cuda_stream);

/* ---------------------------------------------------------------------------
 * Handing the composed map to the consumer (Section 2.2: make an operator's
 * data lie where the next operator needs it, so that no copy runs between
 * them).  amap_map_device_view flattens a map into the plain struct of
 * amap_device.h, which a CUDA kernel takes by value and reads through with
 * amap_view_locate(): the result tensor of the chain is never materialised.
 * Only maps with one stage and one output, at most AMAP_VIEW_MAX_PIECES
 * pieces of at most AMAP_VIEW_MAX_LOOPS loops and AMAP_VIEW_MAX_CONS
 * constraints each, qualify (AMAP_ETOOLARGE / AMAP_EUNSUPPORTED otherwise).
 * `out` is a host pointer to a caller-owned struct; no CUDA call is made.
 * ------------------------------------------------------------------------- */
struct amap_device_view;
int amap_map_device_view(const amap_map *map, struct amap_device_view *out);

/* A demonstration consumer: the sums of the rows of the chain's RESULT, seen as a rows x cols matrix of unsigned
 * integers of elem_size (1, 2 or 4) bytes, added modulo 2^32 -- computed by a kernel that reads the external inputs
 * through the view, without the result ever being written (for an im2col map this is a box filter that touches
 * only the image).  rows * cols must equal the view's out_numel.
 *   view          host pointer (copied into the kernel's parameters)
 *   src_dev_ptrs  host array of the view's n_inputs DEVICE pointers (16-byte aligned)
 *   sums_dev      DEVICE pointer to rows uint32 values
 * Enqueues one kernel on cuda_stream of the current device and returns without synchronising or allocating.
 * Where every row is a whole number of contiguous source runs of one piece (rows of an im2col matrix, of a head
 * split, of a plain copy) the kernel decodes the loops outside a row once per row and takes the runs inside it from
 * a table (amap_device.h: amap_view_rows); otherwise it asks amap_view_locate per 16 bytes. */
int amap_consume_row_sums(const struct amap_device_view *view, const void *const *src_dev_ptrs, int64_t rows,
                          int64_t cols, uint32_t *sums_dev, void *cuda_stream);

/* The row tables of amap_device.h (amap_view_rows_build, amap_view_row_seek, amap_view_row_run) walked on the HOST:
 * writes the chain's result, seen as rows of `cols` elements, to dst_host from HOST copies of the inputs.  For
 * tests of the tables a consumer kernel relies on.  AMAP_EUNSUPPORTED when the rows of the view are not whole runs
 * of one piece each (a consumer then falls back to amap_view_locate); elem_size up to 8. */
int amap_view_rows_gather_host(const struct amap_device_view *view, int64_t cols, const void *const *src_host_ptrs,
                               void *dst_host);

const char *amap_strerror(int code);
/* text of the last CUDA error seen by this thread in this library ("" if none) */
const char *amap_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* AMAP_H_ */
