/*
 * erase.h -- C ABI of the ERASE training-step library for NVIDIA B200 (sm_100a).
 *
 * The library runs one training step of a network cut into B detached blocks, each trained by
 * its own local loss (paper Section 2.1, Eq. 1):
 *
 *     z_0 = x,   z_b = f_b( sg[z_{b-1}] ; theta_b ),   l_b = loss( head_b(z_b), target )
 *
 * sg[] is the stop-gradient: identity going forward, zero Jacobian going backward, so the
 * gradient of theta_b depends on block b alone and is ready as soon as block b's forward and
 * local loss have run.  The step can be enqueued in two orders that give bit-identical results:
 *
 *   serial (n_streams = 1)  F_1 .. F_B, B_B .. B_1, optimizer  on one stream -- the conventional
 *                           forward-then-backward order of Section 2.2, Eq. 2 (all lambda_i = 1,
 *                           no L_main);
 *   ERASE  (n_streams >= 2) F_b on the main stream; a per-block event releases B_b onto side
 *                           stream (b-1) mod (n_streams-1) as soon as F_b and l_b are enqueued, so
 *                           B_b overlaps F_{b+1} (Section 2.2); the optimizer waits on every
 *                           block's backward event.
 *
 * Every pointer in this interface is a HOST pointer unless its comment says DEVICE.  Device
 * pointers must belong to the CUDA device that was current when erase_create() ran.  No call
 * throws or aborts; every failure is reported through the returned status, and a message can be
 * read with erase_last_error().  All calls on one model must come from one host thread at a time.
 */
#ifndef ERASE_H_
#define ERASE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ERASE_API __attribute__((visibility("default")))
#else
#define ERASE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct erase_model erase_model; /* opaque; owned by the library */

typedef enum {
  ERASE_OK = 0,
  ERASE_EINVAL = 1,       /* bad argument or spec; nothing was launched.  Also returned by the
                             first synchronising call after a step whose batch held an id outside
                             its table: the id was not dereferenced, the step's results are void */
  ERASE_ENOMEM = 2,       /* device or host allocation failed, or the caller's arena is small */
  ERASE_ECUDA = 3,        /* a CUDA call failed; text in erase_last_error()                  */
  ERASE_ESTATE = 4,       /* call not valid in this state (e.g. step before parameters set)  */
  ERASE_ETIMEOUT = 5,     /* a bounded device-side wait expired; the step's results are void */
  ERASE_EUNSUPPORTED = 6, /* valid request that this build does not implement                */
  ERASE_ECOMM = 7         /* NCCL could not be loaded, or one of its calls failed            */
} erase_status;

typedef enum { ERASE_F32 = 0, ERASE_BF16 = 1 } erase_dtype;      /* operand/activation precision;
                                                   accumulation, gradients, optimizer are fp32 */
typedef enum { ERASE_IN_DENSE = 0, ERASE_IN_TOKENS = 1, ERASE_IN_CTR = 2 } erase_input_kind;
typedef enum { ERASE_BLK_MLP = 0,         /* Linear act Linear ... (no activation after the last) */
               ERASE_BLK_TOWER = 1,       /* Linear act after every Linear                        */
               ERASE_BLK_TRANSFORMER = 2, /* pre-LN causal transformer block, dims = {d, d_ff}    */
               ERASE_BLK_CROSS = 3,       /* n_cross DCN-v2 layers x_{l+1} = x0 * (W x_l + b) + x_l */
               ERASE_BLK_DOT = 4,         /* dense projection, pairwise dots, then a tower        */
               ERASE_BLK_MAIN = 5         /* last block only: the UNDETACHED remainder of Section 2.2, Eq. 2.  A tower
                                             (activation after every Linear) over u = [z_0 | sg z_1 | .. | sg z_B]
                                             (z_0 only with ERASE_MAIN_READS_INPUT), BCE head, loss L_main.  Its
                                             backward is the usual one: it runs behind the last forward, trains the
                                             tower and -- with train_input -- the input tables through the z_0
                                             columns of u; the sg z_b columns pass nothing back.  dims[0] must be
                                             the width of u.  Dense or CTR input.                              */
} erase_block_kind;
#define ERASE_MAIN_READS_INPUT 1   /* erase_block_spec.flags of a MAIN block: u starts with the undetached z_0 */
typedef enum { ERASE_ACT_NONE = 0, ERASE_ACT_RELU = 1, ERASE_ACT_GELU = 2 } erase_act;
typedef enum { ERASE_HEAD_BCE = 0,        /* Linear(d->1) + mean binary cross-entropy with logits */
               ERASE_HEAD_SOFTMAX_CE = 1, /* Linear(d->head_out) + mean softmax cross-entropy     */
               ERASE_HEAD_GOODNESS = 2    /* Section 2.1: binary cross-entropy on the goodness score
                                             G = sum_j z_j^2; logit G + bh (bh: trainable scalar, minus
                                             the threshold), labels y (1 = positive); no head weights;
                                             head_out = 1; dense or CTR input                     */
} erase_head_kind;
typedef enum { ERASE_OPT_SGD = 0, ERASE_OPT_ADAM = 1, ERASE_OPT_ADAMW = 2 } erase_opt_kind;
typedef enum { ERASE_TOPO_CHAIN = 0,      /* block b reads sg[z_{b-1}] (Eq. 1)                    */
               ERASE_TOPO_PARALLEL = 1    /* every block reads sg[z_0]                            */
} erase_topology;

#define ERASE_MAX_DIMS 8

/* One detached block f_b together with its local head (Section 2.1). */
typedef struct {
  int32_t kind;                 /* erase_block_kind                                              */
  int32_t n_dims;               /* entries used in dims                                          */
  int32_t dims[ERASE_MAX_DIMS]; /* MLP/TOWER: layer widths d0..dL; TRANSFORMER: {d_model, d_ff};
                                   CROSS: {width}; DOT: {padded feature count, tower widths...}   */
  int32_t act;                  /* erase_act between (MLP) / after (TOWER, DOT) the Linears;
                                   TRANSFORMER always uses exact-erf GELU, CROSS none             */
  int32_t n_heads;              /* TRANSFORMER: attention heads; head width must be 64 or a
                                   divisor of d_model with d_model/n_heads <= 128                */
  int32_t n_cross;              /* CROSS: number of cross layers                                 */
  int32_t head;                 /* erase_head_kind                                               */
  int32_t head_out;             /* 1 for BCE; vocabulary size for softmax cross-entropy          */
  int32_t flags;                /* MAIN: ERASE_MAIN_READS_INPUT; 0 otherwise                     */
} erase_block_spec;

/* The whole model.  Trainable tensors are Linear weights W [out, in] row-major, biases, and
 * LayerNorm gain/shift; the input tables (token/position embeddings, CTR tables) sit under
 * sg[z_0] and are frozen. */
typedef struct {
  int32_t dtype;      /* erase_dtype                                                             */
  int32_t input;      /* erase_input_kind                                                        */
  int32_t topo;       /* erase_topology                                                          */
  int32_t batch;      /* samples per step (sequences for TOKENS)                                 */
  int32_t width;      /* DENSE: input width; TOKENS: d_model; CTR: packed width of x0            */
  int32_t seq;        /* TOKENS: sequence length T (targets are the inputs shifted by one)       */
  int32_t vocab;      /* TOKENS: vocabulary size                                                 */
  int32_t n_dense;    /* CTR: dense features per sample                                          */
  int32_t n_sparse;   /* CTR: sparse features (= embedding tables), one id each                  */
  int32_t table_rows; /* CTR: rows per table                                                     */
  int32_t emb_dim;    /* CTR: embedding width                                                    */
  int32_t n_blocks;
  const erase_block_spec* blocks; /* n_blocks entries; copied by erase_create                    */
  int32_t opt;        /* erase_opt_kind                                                          */
  float lr, beta1, beta2, eps, weight_decay; /* Adam: m,v with bias correction, update
                         lr*mhat/(sqrt(vhat)+eps); AdamW first shrinks theta by (1 - lr*wd)      */
  int32_t train_input; /* CTR with a MAIN block that reads z_0: the embedding tables are trained by L_main
                         (gradient = scatter-add of dL_main/dz_0 by id, summed in sample order; the
                         optimizer touches only the rows the batch read; untouched rows keep their
                         values and moments).  Tables then count as trainable tensors: erase_grads
                         returns their dense gradient of the last step, erase_opt_state their moments.
                         batch <= 16384.                                                           */
  int32_t replicas;   /* data-parallel replicas that train this model together (0 and 1: this model alone).
                         Each replica steps on its own `batch` samples; every local loss is the mean over
                         all replicas * batch samples, so a replica's own losses and gradients are its
                         share of the sums (see erase_comm_init).                                 */
  void* arena;        /* DEVICE, optional: caller-owned memory the model lives in (256-byte
                         aligned); NULL = the library allocates with cudaMalloc                  */
  size_t arena_bytes; /* size of arena; at least erase_arena_bytes(spec)                         */
} erase_model_spec;

/* One batch, all DEVICE pointers, owned by the caller and kept alive and unmodified until the
 * step has been synchronised (erase_sync / erase_losses).
 *   DENSE : x [batch, width] row-major in the model dtype (float or bfloat16 bits); y [batch] float
 *   TOKENS: ids [batch, seq+1] int32 in [0, vocab); inputs are ids[:, :seq], targets ids[:, 1:]
 *   CTR   : x = dense features [batch, n_dense] float; ids [batch, n_sparse] int32 in
 *           [0, table_rows); y [batch] float.  x0 = [table_t[ids[n,t]] for t | dense | zero pad]. */
typedef struct {
  const void* x;
  const int32_t* ids;
  const float* y;
} erase_batch;

/* erase_step_ex flags */
#define ERASE_GRAPH 1u   /* replay the whole step (either schedule) as one CUDA graph, captured on
                            first use per (batch pointers, n_streams, flags); Section 1.1/2.2      */
#define ERASE_NO_OPT 2u  /* stop after the backward passes: gradients only, parameters untouched   */
#define ERASE_EARLY_HEAD 4u /* ERASE schedules only: release the side stream right after the block
                            BODY's forward and run the local head, its loss and the backward there.
                            The next block's forward needs z_b but not l_b, so the head leaves the
                            main stream's critical path (Section 2.1: the gradient is ready once
                            forward and local loss are done -- nothing else waits for the loss).
                            Same kernels, same bits.  Without the flag the head and loss run on the
                            main stream before the release, as the paper schedules them.          */

#define ERASE_BLOCK_OPT 8u /* ERASE schedules only: update theta_b on block b's side stream right after
                            B_b instead of in one sweep after every backward has finished.  theta_b is
                            read by F_b and B_b alone (Section 2.1: the gradient of block b is final
                            once B_b ends), so the optimizer's serial tail disappears under the other
                            blocks' work.  Same update kernel on the same values: same bits.          */

#define ERASE_SPLIT_BWD 16u /* ERASE schedules only: inside B_b, the operations that only produce a
                            parameter gradient (weight-gradient GEMMs and their reductions, bias column
                            sums, LayerNorm gain/shift gradients) run on a second stream per block,
                            each released by an event behind the gradient-chain operation whose output
                            it reads; the chain (dgrads, attention, LayerNorm dx) stays on the block's
                            side stream and the two join before the block's optimizer.  Nothing in B_b
                            reads a parameter gradient, and every backward buffer is written once per
                            step, so this is the overlap of Section 2.2 applied one level down.  Same
                            kernels on the same values: same bits.                                    */

#define ERASE_STAMPS 32u  /* record the phase timeline of this step with device clock stamps (a one-thread
                            kernel per phase boundary) instead of CUDA events, which cannot be captured:
                            with ERASE_GRAPH the stamps are part of the graph, and erase_timeline then
                            shows how the phases of a REPLAYED step overlap.  A measuring aid: it adds
                            2*(2*n_blocks+1)+1 tiny kernels to the step.                               */

#define ERASE_PAR_FWD 64u /* ERASE schedules on the PARALLEL topology only (every block reads z_0; ignored
                            on chains): the blocks' forwards do not depend on one another either, so
                            block b's whole chain F_b, l_b, B_b (and, with ERASE_BLOCK_OPT, its
                            optimizer) runs on its side stream, released by one event behind the input
                            staging: up to n_streams-1 blocks train side by side.  Wider than the
                            paper's overlap of B_b with F_{b+1} (Section 2.2); same kernels, same bits. */

#define ERASE_PERSISTENT 128u /* co-schedule F_{b+1} and B_b inside ONE persistent kernel on a partition of the SMs
                            (Section 2.2: B_b overlaps F_{b+1}; Sections 1 and 3.1: small GEMMs leave SMs idle and
                            can share the device).  The step runs on the main stream alone, n_streams is
                            ignored: stage s launches one dual-list kernel whose first share of the CTAs works
                            through the GEMMs and GELU passes of F_s and the rest through those of B_{s-1}, each
                            list in order with device-side completion counters between dependent problems; the
                            heads, losses, reductions and the optimizer stay ordinary launches between stages.
                            Same tile arithmetic in the same order: same bits as the serial schedule.  Available
                            for bf16 chains of MLP / tower blocks (the saturation-sweep models); other models get
                            ERASE_EUNSUPPORTED with the reason in erase_last_error().  May be combined with
                            ERASE_GRAPH and ERASE_NO_OPT; the stream-placement flags are ignored.          */

#define ERASE_LOCAL_GRADS 256u /* step without the exchange between replicas: losses and gradients stay this
                            replica's share of the global sums (they add up, over the replicas, to the
                            losses and gradients of one model on the union of the batches).  For callers
                            that exchange gradients themselves, usually with ERASE_NO_OPT, and for
                            accumulating a large batch in pieces.  The only way to step a model built
                            with replicas > 1 that has no communicator.                               */

/* Device bytes erase_create needs for this spec when given an arena; 0 if the spec is invalid. */
ERASE_API size_t erase_arena_bytes(const erase_model_spec* spec);

/* Builds the model on the current CUDA device: validates the spec, lays out parameters,
 * gradients, optimizer state, per-block activation stashes and scratch, creates streams and
 * events.  Parameters start undefined: set every tensor with erase_set_params before stepping.
 * On failure *out is untouched.  Errors: EINVAL (spec), ENOMEM, ECUDA. */
ERASE_API erase_status erase_create(const erase_model_spec* spec, erase_model** out);

/* Waits for outstanding work, frees everything the library allocated.  NULL is allowed. */
ERASE_API void erase_destroy(erase_model* m);

/* Tensor table.  Order: frozen input tables first (tok_emb, pos_emb | table0..), then block by
 * block: MLP/TOWER W0,b0,W1,b1,..; TRANSFORMER ln1_g,ln1_b,Wqkv,bqkv,Wproj,bproj,ln2_g,ln2_b,
 * W1,b1,W2,b2; CROSS Wc0,bc0,..; DOT Wd,bd,W0,b0,..; each block ends with its head Wh,bh (the
 * goodness head: bh only). */
ERASE_API int32_t erase_num_tensors(const erase_model* m);
/* block = -1 for frozen input tables; name receives a NUL-terminated string (<= 31 chars);
 * shape has rank entries (<= 2).  Errors: EINVAL (index, NULL). */
ERASE_API erase_status erase_tensor_info(const erase_model* m, int32_t idx, int32_t* block, char name[32],
                               int32_t* rank, int64_t shape[4], int32_t* trainable);

/* Parameters travel as fp32 host arrays of exactly n = product(shape) elements.
 * set: copies into the fp32 master (and refreshes the bf16 operand copy); synchronous.
 * params/grads: wait for the last enqueued step, then copy out.  grads are those of the last
 * step (d l_b / d theta_b, fp32).  Errors: EINVAL (index, size, NULL, frozen tensor for grads). */
ERASE_API erase_status erase_set_params(erase_model* m, int32_t idx, const float* src, size_t n);
ERASE_API erase_status erase_params(erase_model* m, int32_t idx, float* dst, size_t n);
ERASE_API erase_status erase_grads(erase_model* m, int32_t idx, float* dst, size_t n);

/* Adam moments of one trainable tensor and the global step counter t (number of optimizer
 * steps taken).  Any of mom1/mom2/t may be NULL.  With SGD the moments read as zeros. */
ERASE_API erase_status erase_opt_state(erase_model* m, int32_t idx, float* mom1, float* mom2, size_t n, int64_t* t);
ERASE_API erase_status erase_set_opt_state(erase_model* m, int32_t idx, const float* mom1, const float* mom2,
                                 size_t n, int64_t t);

/* Enqueues one training step on the model's streams and returns without waiting.
 * n_streams = 1: serial schedule; n_streams >= 2: ERASE with n_streams-1 side streams (values
 * above n_blocks+1 are clamped).  erase_step(m,b,n) == erase_step_ex(m,b,n,0).
 * Errors: EINVAL (NULL, missing batch pointer, n_streams < 1), ESTATE (a tensor was never set),
 * ECUDA. */
ERASE_API erase_status erase_step(erase_model* m, const erase_batch* batch, int32_t n_streams);
ERASE_API erase_status erase_step_ex(erase_model* m, const erase_batch* batch, int32_t n_streams, uint32_t flags);

/* Waits for the last step and copies the local losses l_1..l_B (n_blocks floats; a MAIN block is the
 * last of them and its entry is L_main) to dst. */
ERASE_API erase_status erase_losses(erase_model* m, float* dst, int32_t n_blocks);

/* Waits until everything enqueued on the model has finished. */
ERASE_API erase_status erase_sync(erase_model* m);

/* Checks the library's time-out path without any real failure: enqueues, on the model's main
 * stream, ONE thread that waits on a barrier nothing will ever signal -- with the same bounded
 * wait the GEMM kernels use, limited to about limit_us microseconds (1..100000) -- then records
 * the expiry in the model's status word and returns.  Nothing hangs and nothing faults: the wait
 * is bounded by the SM clock.  The next erase_sync / erase_losses / erase_params returns
 * ERASE_ETIMEOUT and clears the word; tensor-core kernels enqueued in between find the word set and
 * skip their work, so a step behind an expired wait costs one limit, not one per kernel.  The
 * model stays usable afterwards.  (Section 2.2 synchronises with streams and events only; the
 * barriers inside the tensor-core kernels are this library's own, hence this check.)
 * Errors: EINVAL, ECUDA. */
ERASE_API erase_status erase_selftest_timeout(erase_model* m, int32_t limit_us);

/* Data-parallel replicas (Section 3: the CTR model is trained on eight GPUs with gradient
 * synchronisation between them; Sections 2.2 and 4: once backward passes leave the main stream, every
 * rank must still issue its collectives in one and the same order, or ranks wait on one another).
 * One process per GPU holds one replica built from the
 * same spec (replicas = world) and the same parameters.  A step then is: every replica runs F_b, l_b and
 * B_b on its own batch; right behind B_b, on the stream B_b ran on, block b's slice of the fp32
 * gradient arena is summed over the replicas in place (one NCCL all-reduce per block, so the exchange of
 * block b overlaps F_{b+1..} exactly as B_b does); the B local losses are summed the same way at the
 * join; the optimizer (of the block, with ERASE_BLOCK_OPT; else the sweep) follows the exchange, so every
 * replica applies the same update to the same values and the replicas stay bit-identical to one
 * another.  The order of the exchanges depends only on (n_streams, flags): pass the same to every replica.
 *
 * erase_comm_unique_id: fills 128 HOST bytes with a fresh NCCL id; call on one replica and carry the
 *   bytes to the others by any means (a file, a socket, torch.distributed).
 * erase_comm_init: id = those 128 bytes (HOST).  Collective over the replicas (blocks until all have called
 *   it, as ncclCommInitRank does); the current CUDA device must be the model's.  world must equal the
 *   spec's replicas (1 is allowed: a communicator of one, the exchange then changes nothing).  The
 *   communicator lives until erase_destroy.
 * erase_comm_order: the block index of every exchange the last step enqueued, in enqueue order
 *   (-1 stands for the losses), at most cap entries into blocks_out (HOST); *n_out = their number.  Serial schedule:
 *   B-1, .., 0, -1; ERASE: 0, .., B-1, -1.
 * NCCL is loaded when first needed ("libnccl.so.2", or the file the environment variable
 * ERASE_NCCL_LIB names).  A replica that stops stepping leaves the others waiting inside NCCL: the
 * library adds no watchdog of its own.  Not offered with a communicator attached: ERASE_GRAPH, and
 * train_input with world > 1 (sparse table gradients are not exchanged).
 * Errors: EINVAL, ESTATE (a communicator is attached already), EUNSUPPORTED, ECOMM, ECUDA. */
#define ERASE_COMM_ID_BYTES 128
ERASE_API erase_status erase_comm_unique_id(void* id_out);
ERASE_API erase_status erase_comm_init(erase_model* m, int32_t rank, int32_t world, const void* id);
ERASE_API erase_status erase_comm_order(erase_model* m, int32_t* blocks_out, int32_t cap, int32_t* n_out);

/* The CUDA stream (cudaStream_t) that steps start and end on; valid until erase_destroy.  A
 * caller may record its own events on it to time steps. */
ERASE_API void* erase_main_stream(erase_model* m);

/* Kernels launched by this library on behalf of the model since it was created. */
ERASE_API int64_t erase_launch_count(const erase_model* m);

/* Device-side begin/end times of the last step's phases, in milliseconds relative to the step's
 * start, from CUDA events: out[2*b], out[2*b+1] = start and end of F_b for b < n_blocks, then
 * the same for B_b, then for the optimizer: 2*(2*n_blocks+1) floats.  Recorded for steps run
 * without ERASE_GRAPH (CUDA events) and for steps run with ERASE_STAMPS (device clock stamps,
 * graph replay included).  With ERASE_BLOCK_OPT the optimizer entries bracket the join only.
 * Waits for the step.  Errors: EINVAL, ESTATE (no such step). */
ERASE_API erase_status erase_timeline(erase_model* m, float* out, int32_t n);

/* The GEMM the block linears are made of, on its own (paper Section 1: the "small GEMMs" of proxy
 * models are where the accelerator's capacity goes unused).  C[M,N] = sum_k A(m,k) B(n,k) with
 * A(m,k) = A[m*sa_m + k*sa_k] and B(n,k) = B[n*sb_n + k*sb_k] (element strides; one stride of
 * each operand must be 1), so the same call covers X W^T (forward), dY W (dgrad, B strided over
 * k) and dY^T X (wgrad, both strided over k).  A, B, C are DEVICE pointers; dtype selects float
 * or bfloat16 operands; C is float when c_f32 != 0, else the operand type, row stride ldc.
 * splits > 1 runs a deterministic split-K (fixed partition, partial sums added in order).
 * engine: 0 = SIMT kernel, 1 = tcgen05 tensor-core kernel (bf16 only; EUNSUPPORTED when the
 * shape or alignment does not qualify: K >= 64, N >= 16, 16-byte aligned bases, leading strides
 * multiples of 8).  The call allocates its split-K workspace, runs on `stream` (a cudaStream_t,
 * may be NULL for the default stream), waits for completion and frees the workspace.
 * Errors: EINVAL, ENOMEM, EUNSUPPORTED, ECUDA, ETIMEOUT (a bounded device wait expired). */
ERASE_API erase_status erase_gemm(int32_t dtype, int32_t M, int32_t N, int32_t K, const void* A, int64_t sa_m,
                                  int64_t sa_k, const void* B, int64_t sb_n, int64_t sb_k, void* C, int64_t ldc,
                                  int32_t c_f32, int32_t splits, int32_t engine, void* stream);

/* erase_gemm for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a deployment convenience of the library, not part of the method.)
 *
 * Who needs it: code running inside a process whose device memory is entirely managed by
 * someone else's pool, code on a latency budget that cannot afford the device-wide
 * synchronisation a cudaMalloc/cudaFree may imply, and code called at moments when allocation is
 * forbidden.  Same arguments, semantics and results as erase_gemm, but the split-K workspace and
 * the status word live in one fixed array inside the library's device image
 * (ERASE_STATIC_WS_FLOATS floats, 8 MiB, plus 256 bytes; every GPU that loads the library holds
 * it until the process exits).  The call performs no cudaMalloc, cudaFree or other allocating
 * call, here or in any library.
 *   - splits*M*N must not exceed ERASE_STATIC_WS_FLOATS (only when splits > 1); larger
 *     requests are refused with EINVAL and a message naming the limit.  Nothing is launched.
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current).  Make that first call outside any CUDA stream capture.
 *   - All calls on a device share the array and it keeps the last call's contents; the call
 *     clears what must start at zero itself.  Two calls whose GPU work overlaps in time (different
 *     streams or threads) race on it: issue them one after the other.
 * The text of this entry point's last error on the calling thread: erase_gemm_static_error(). */
#define ERASE_STATIC_WS_FLOATS (2u * 1024u * 1024u)
ERASE_API erase_status erase_gemm_static(int32_t dtype, int32_t M, int32_t N, int32_t K, const void* A,
                                         int64_t sa_m, int64_t sa_k, const void* B, int64_t sb_n, int64_t sb_k,
                                         void* C, int64_t ldc, int32_t c_f32, int32_t splits, int32_t engine,
                                         void* stream);
ERASE_API const char* erase_gemm_static_error(void);

/* One record per operation of a profiled step. */
typedef struct {
  char name[32];    /* kernel class: gemm_fwd, gemm_dgrad, gemm_wgrad, softmax_ce, opt_update, ...   */
  int32_t block;    /* block index, -1 for input staging and the optimizer                         */
  int32_t phase;    /* 0 input staging, 1 forward F_b, 2 backward B_b, 3 optimizer                  */
  int32_t launches; /* kernels this operation launches                                             */
  float ms;         /* device time between CUDA events recorded around the operation               */
  double flops;     /* algorithmic floating-point operations (2*M*N*K for a GEMM)                  */
  double bytes;     /* algorithmic bytes: every operand read once, every result written once       */
} erase_op_record;

/* Runs one complete step in the serial order on the main stream with a pair of CUDA events around
 * every operation, waits for it, and writes one record per operation to out (at most cap; *n
 * receives the number of operations the step has).  It is a real step: parameters are updated.
 * Used to attribute time to kernels (the roofline of the dominant kernel); the event pairs
 * serialise nothing but add launch gaps, so whole-step time is NOT measured here.
 * Errors: as erase_step, and EINVAL for NULL out/n. */
ERASE_API erase_status erase_profile_step(erase_model* m, const erase_batch* batch, erase_op_record* out,
                                          int32_t cap, int32_t* n);

/* Text of the last error on this model ("" if none); NULL model gives the text of the last
 * failed erase_create on this thread. */
ERASE_API const char* erase_last_error(const erase_model* m);

#ifdef __cplusplus
}
#endif
#endif /* ERASE_H_ */
