/*
 * splitlora.h -- C ABI of the B200 (sm_100a) split-LoRA round library.
 *
 * One training round t of SplitLoRA (arxiv 2407.00952, Algorithm 1) on a GPT-style pre-LN decoder
 * cut after block `cut`:
 *   splitlora_client_fwd   step a1/a2, Eq. 2 : K clients run blocks 1..cut, each with its own adapters
 *   splitlora_server_step  step a3/a4, Eq. 3-5: server forward + loss + backward + server update
 *   splitlora_client_bwd   step a5, Eq. 6-7  : activation gradients back through the client blocks + update
 *   splitlora_aggregate    stage b, Eq. 8-9  : data-size-weighted average of the client A and B matrices
 *   splitlora_round        one iteration of Algorithm 1 (the four calls above; aggregation every I rounds)
 *
 * General rules
 *   - Every function returns 0 (SPLITLORA_OK) or a negative error code; nothing throws, exits or
 *     falls back to the CPU.  splitlora_last_error() gives a text for the last failure of a context.
 *   - Unless a parameter is marked HOST it is a DEVICE pointer, 16-byte aligned, contiguous,
 *     row-major, owned by the caller and only borrowed (frozen weights and the workspace for the
 *     life of the context, everything else for the duration of the call).
 *   - Work is enqueued on the CUDA stream given at creation; calls return without synchronising
 *     unless they write to a HOST pointer (loss_out).
 *   - The library never allocates device memory in the calls below: all of its state lives in the
 *     caller-provided workspace (splitlora_workspace_bytes / splitlora_bind_workspace).
 *   - A process may use several devices: per-device set-up (kernel attributes, SM count, status
 *     words) is keyed by the device that is current when a call is made, so make the context's
 *     device current before every call on that context.
 *   - Conventions: a linear layer stores W as [out, in]; a LoRA adapter is A [r, in], B [out, r]
 *     and the adapted layer computes  y = x W^T + bias + (alpha/r) (x A^T) B^T   (Sec. II-C).
 *     Activations are [K, b, T, d] = [clients, sequences per client, positions, width].
 */
#ifndef SPLITLORA_H_
#define SPLITLORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPLITLORA_OK              0
#define SPLITLORA_ERR_ARG        -1   /* null pointer, out-of-range or inconsistent argument        */
#define SPLITLORA_ERR_ALIGN      -2   /* a device pointer is not 16-byte aligned                    */
#define SPLITLORA_ERR_STATE      -3   /* call order (e.g. client_bwd without client_fwd, unbound weights) */
#define SPLITLORA_ERR_ARCH       -4   /* the current device is not compute capability 10.x          */
#define SPLITLORA_ERR_WORKSPACE  -5   /* workspace missing or too small                             */
#define SPLITLORA_ERR_COUNTS     -6   /* a negative sample count, or all counts zero                */
#define SPLITLORA_ERR_TIMEOUT    -7   /* a bounded wait inside a kernel expired (see device_status) */
#define SPLITLORA_ERR_CUDA       -8   /* a CUDA call failed; text in splitlora_last_error           */
#define SPLITLORA_ERR_UNSUPPORTED -9  /* a valid request that this build does not implement         */

#define SPLITLORA_DTYPE_FP32 0        /* everything fp32 (plain FMA arithmetic, no tensor cores)    */
#define SPLITLORA_DTYPE_BF16 1        /* bf16 activations + frozen tensors, fp32 accumulation, fp32 adapters */

#define SPLITLORA_OPT_SGD   0         /* Eq. 4-7 literally: P <- P - gamma G                        */
#define SPLITLORA_OPT_ADAMW 1         /* AdamW with bias correction and decoupled weight decay      */

#define SPLITLORA_TARGET_Q 1u         /* bits of lora_targets: which slices of the fused qkv        */
#define SPLITLORA_TARGET_K 2u         /* projection carry an adapter                                */
#define SPLITLORA_TARGET_V 4u
#define SPLITLORA_TARGET_O 8u         /* the attention output projection                            */

#define SPLITLORA_ARCH_GPT   0        /* LayerNorm, learned positions, GELU MLP, biases, head tied to
                                         wte: the paper's GPT-2 (Sec. IV-A)                          */
#define SPLITLORA_ARCH_LLAMA 1        /* RMSNorm, rotary positions on q and k (pairs j, j + dh/2),
                                         SwiGLU MLP, no biases, separate head.  The paper cites
                                         Llama-2 only as an LLM and does not describe this shape    */

#define SPLITLORA_SIDE_CLIENT 0
#define SPLITLORA_SIDE_SERVER 1

typedef struct splitlora_ctx splitlora_ctx;   /* opaque */

/* Inputs of Algorithm 1 (b, I, gamma_c, gamma_s, N) plus the model shape.  Plain data. */
typedef struct {
  int32_t n_layer;           /* blocks in the whole model                                   */
  int32_t cut;               /* blocks 0..cut-1 run on the clients; 1 <= cut <= n_layer.
                                cut == n_layer: every block is client-side and aggregated,
                                the server keeps only the final norm and the head (the
                                federated-LoRA baseline of Sec. IV-A); n_clients == 1 is
                                the centralised baseline                                    */
  int32_t d_model, n_head, d_ff, vocab, max_seq;
  int32_t lora_r;            /* rank r, 1..64                                               */
  float   lora_alpha;        /* scaling alpha; the update is scaled by alpha / r            */
  uint32_t lora_targets;     /* SPLITLORA_TARGET_* bits                                     */
  int32_t n_clients;         /* K (the paper's N)                                           */
  int32_t batch_per_client;  /* b                                                           */
  int32_t seq;               /* T <= max_seq                                                */
  int32_t dtype;             /* SPLITLORA_DTYPE_*                                           */
  int32_t optimizer;         /* SPLITLORA_OPT_*                                             */
  float   lr_client, lr_server;          /* gamma_c, gamma_s                                */
  float   beta1, beta2, adam_eps, weight_decay;
  int32_t agg_interval;      /* I: aggregate when round_index % I == 0, round_index from 1  */
  float   norm_eps;
  int32_t gelu_tanh;         /* 1: tanh form of GELU (GPT-2), 0: erf form                   */
  int32_t use_tensor_cores;  /* bf16 only: 1 = tcgen05 GEMMs + tensor-core attention (default),
                                0 = plain FMA kernels (a second opinion for debugging)      */
  int32_t arch;              /* SPLITLORA_ARCH_*                                            */
  float   rope_theta;        /* base of the rotary frequencies (ARCH_LLAMA only), e.g. 1e4  */
  int32_t cut_min;           /* 0: every client is cut at `cut`.  Else 1 <= cut_min <= cut: clients
                                may be cut at different depths in [cut_min, cut] (see
                                splitlora_set_client_cuts); client adapters are stored for blocks
                                0..cut-1 and the server has adapters on blocks cut_min..n_layer-1 */
} splitlora_config;

/* ---- context ------------------------------------------------------------------------------ */

/* Validates cfg (HOST), checks the device, records `cuda_stream` (a cudaStream_t, may be NULL for
 * the default stream).  *out is owned by the caller until splitlora_destroy. */
int splitlora_create(const splitlora_config* cfg, void* cuda_stream, splitlora_ctx** out);
int splitlora_destroy(splitlora_ctx* ctx);

/* Bytes of device memory the context needs for saved activations, adapters, optimizer state,
 * transposed frozen copies and scratch.  bytes is HOST. */
int splitlora_workspace_bytes(const splitlora_config* cfg, size_t* bytes);
/* Gives the context its workspace (256-byte aligned).  Initialises adapters to zero, optimizer
 * state to zero, round counter to 0. */
int splitlora_bind_workspace(splitlora_ctx* ctx, void* dev, size_t bytes);

/* Frozen tensors of W_c and W_s, in the context dtype.  Names (l = block index from 0):
 *   "wte" [vocab, d]   "wpe" [max_seq, d]   "lnf.g" [d]   "lnf.b" [d]
 *   "h.<l>.ln1.g" "h.<l>.ln1.b" [d]          "h.<l>.attn.qkv.w" [3d, d]  "h.<l>.attn.qkv.b" [3d]
 *   "h.<l>.attn.proj.w" [d, d] "h.<l>.attn.proj.b" [d]   "h.<l>.ln2.g" "h.<l>.ln2.b" [d]
 *   "h.<l>.mlp.fc1.w" [d_ff, d] "h.<l>.mlp.fc1.b" [d_ff] "h.<l>.mlp.fc2.w" [d, d_ff] "h.<l>.mlp.fc2.b" [d]
 * The LM head is tied to "wte".  With ARCH_LLAMA the set is instead
 *   "wte" [vocab, d]   "head.w" [vocab, d]   "lnf.g" [d]
 *   "h.<l>.ln1.g" [d]  "h.<l>.attn.qkv.w" [3d, d]  "h.<l>.attn.proj.w" [d, d]  "h.<l>.ln2.g" [d]
 *   "h.<l>.mlp.gate_up.w" [2*d_ff, d] (rows 0..d_ff-1 gate, the rest up)  "h.<l>.mlp.down.w" [d, d_ff]
 * Tensors are borrowed and never written.  `bytes` must equal the
 * size implied by the shape.  Requires a bound workspace (transposed copies for the backward
 * products are made at bind time, on the context stream). */
int splitlora_bind_frozen(splitlora_ctx* ctx, const char* name, const void* dev, size_t bytes);

/* Adapter access (fp32).  side: SPLITLORA_SIDE_*; client: 0..K-1 (ignored for the server);
 * layer: block index (0..cut-1 for clients, cut..n_layer-1 for the server; with cut_min > 0 the
 * server's blocks start at cut_min); target: one
 * SPLITLORA_TARGET_* bit.  A [r, d], B [d, r] device buffers; copied in / out on the stream.
 * Either pointer may be NULL to skip that matrix. */
int splitlora_set_adapter(splitlora_ctx* ctx, int side, int client, int layer, uint32_t target,
                          const float* A, const float* B);
int splitlora_get_adapter(splitlora_ctx* ctx, int side, int client, int layer, uint32_t target,
                          float* A, float* B);
/* Gradients G_A, G_B of the last backward pass (Eq. 4-7), same addressing. */
int splitlora_get_adapter_grad(splitlora_ctx* ctx, int side, int client, int layer, uint32_t target,
                               float* dA, float* dB);
/* AdamW first/second moments, same addressing; for checkpoint / resume. */
int splitlora_get_opt_state(splitlora_ctx* ctx, int side, int client, int layer, uint32_t target,
                            float* mA, float* vA, float* mB, float* vB);
int splitlora_set_opt_state(splitlora_ctx* ctx, int side, int client, int layer, uint32_t target,
                            const float* mA, const float* vA, const float* mB, const float* vB);
/* Round counter t and optimizer step counters (HOST out / in); for resume. */
int splitlora_get_counters(splitlora_ctx* ctx, int64_t* round_index, int64_t* server_steps, int64_t* client_steps);
int splitlora_set_counters(splitlora_ctx* ctx, int64_t round_index, int64_t server_steps, int64_t client_steps);

/* ---- the round (Algorithm 1) -------------------------------------------------------------- */

/* Step a1, Eq. 2.  tokens [K, b, T] int32 in [0, vocab).  Writes the cut-layer activations
 * s_1..s_K to act_out [K, b, T, d] (context dtype): the hand-off buffer of step a2.  Keeps what
 * client_bwd needs inside the workspace. */
int splitlora_client_fwd(splitlora_ctx* ctx, const int32_t* tokens, void* act_out);

/* Step a3/a4, Eq. 3-5.  act_in [K, b, T, d] is treated as the concatenation S^t; labels [K, b, T]
 * int32; a label outside [0, vocab) marks an ignored position (it adds nothing to the loss, to the
 * gradients or to the count the mean is taken over).  One forward/backward over the concatenated batch with the
 * single server adapter set, loss = mean cross-entropy over valid positions, server adapters
 * updated with lr_server.  Writes dL/dS to act_grad_out [K, b, T, d] (context dtype).
 * loss_out is HOST and may be NULL; when given, the call synchronises the stream. */
int splitlora_server_step(splitlora_ctx* ctx, const void* act_in, const int32_t* labels,
                          void* act_grad_out, float* loss_out);

/* Step a5, Eq. 6-7.  Back-propagates act_grad_in [K, b, T, d] through each client's blocks and
 * updates each client's adapters with lr_client.  Needs the saved state of the preceding
 * splitlora_client_fwd on this context, else SPLITLORA_ERR_STATE. */
int splitlora_client_bwd(splitlora_ctx* ctx, const void* act_grad_in);

/* Stage b, Eq. 8-9 and the downlink b3.  sample_counts is HOST int64 [K] (|D_i|), all >= 0 and not
 * all zero.  Every client A and B becomes sum_i (|D_i|/|D|) P_i, written back to all K clients. */
int splitlora_aggregate(splitlora_ctx* ctx, const int64_t* sample_counts);

/* Clients with different adapter ranks (Sec. V, heterogeneous configuration: named as a direction,
 * no rule given).  ranks: HOST int32[K], 1 <= ranks[i] <= lora_r, or NULL to return to one rank for
 * all.  Every client stays stored at lora_r; rank components >= ranks[i] of client i (rows of A,
 * columns of B, and their optimizer moments) are set to zero now and stay zero: their gradients are
 * exactly zero.  The scaling stays alpha / lora_r for every client.  Aggregation applies Eq. 8-9 to
 * these zero-padded matrices (a client without a component adds nothing to it) and each client keeps
 * its own leading ranks[i] components of the average.  Call after the adapters have been set.
 * Errors: SPLITLORA_ERR_ARG (rank out of range), SPLITLORA_ERR_WORKSPACE. */
int splitlora_set_client_ranks(splitlora_ctx* ctx, const int32_t* ranks);

/* Clients cut at different depths (Sec. V, heterogeneous configuration: the joint choice of cut layers
 * and ranks per client is named as a direction, no rule is given).  cuts: HOST int32[K] with
 * cut_min <= cuts[i] <= cut, non-decreasing in i (order the clients by depth), or NULL to return to one
 * cut for all.  Client i then runs blocks 0..cuts[i]-1 with its own adapters and hands off at that
 * depth (row block i of the hand-off buffers is s_i, resp. dL/ds_i, at depth cuts[i]); the server
 * takes client i's rows in at block cuts[i], so the batch of a server block is the clients that have
 * handed off by then, with the server adapters of blocks cut_min..n_layer-1; there is still one loss
 * (mean over all valid positions of all clients) and one server update per round.  Aggregation
 * applies Eq. 8-9 per block to the clients that hold the block, w_i = |D_i| / sum over those holders;
 * a block held by one client is left as it is.  Adapter access for a client is limited to its own
 * blocks.  Needs a configuration with cut_min > 0.  Not available together with clients spread over
 * devices.  Errors: SPLITLORA_ERR_ARG (range, order), SPLITLORA_ERR_WORKSPACE. */
int splitlora_set_client_cuts(splitlora_ctx* ctx, const int32_t* cuts);

/* One iteration t of Algorithm 1: client_fwd, server_step, client_bwd (through internal hand-off
 * buffers) and, when t % agg_interval == 0, aggregate.  tokens, labels DEVICE [K, b, T] int32;
 * sample_counts HOST; loss_out HOST or NULL. */
int splitlora_round(splitlora_ctx* ctx, const int32_t* tokens, const int32_t* labels,
                    const int64_t* sample_counts, float* loss_out);

/* One full t of Algorithm 1 like splitlora_round, with the two tensors that cross the cut handed off
 * compressed (format: see splitlora_handoff_quantize): S after the client forward and dL/dS after the
 * server step are each replaced by codes + scales, and the receiving side continues from the restored
 * values.  codes: device, [2][M, d] bytes (S first, then dL/dS), 16-byte aligned; scales: device,
 * [2][M] fp32; both caller-owned and left holding what the links would carry (M = K*b*T tokens).
 * Everything else (tokens, labels, sample_counts, loss_out_host, errors) as splitlora_round. */
int splitlora_round_compressed(splitlora_ctx* ctx, const int32_t* tokens, const int32_t* labels,
                               const int64_t* sample_counts, uint8_t* codes, float* scales,
                               float* loss_out_host);
/* Same round with HOST tokens and labels: copies them to the device on the stream first.  This is
 * the end-to-end call (host in, host loss out). */
int splitlora_round_host(splitlora_ctx* ctx, const int32_t* tokens_host, const int32_t* labels_host,
                         const int64_t* sample_counts, float* loss_out);

/* ---- sharding the clients of a round over several devices ----------------------------------
 * Clients are independent on the client side (step a1, a5) and the server loss is a mean over the
 * concatenated batch (step a3), so a device can own a subset of the clients and the matching rows
 * of S^t.  Every device holds the same frozen weights and the same server adapters and runs the
 * three calls on its own clients; two sums over devices make the result equal to the one-device
 * round: the server adapter gradients before the server update, and the weighted adapter sum of
 * Eq. 8-9 (one client's worth of parameters) at aggregation.  The library does no communication itself; the caller reduces the
 * buffers below (e.g. with an NCCL all-reduce on the context stream). */

/* Number of valid label positions of the WHOLE concatenated batch (all devices).  When > 0 it
 * replaces the local count as the normaliser of the loss and of dL/dlogits in server_step, so that
 * local losses and gradients add up to the global ones.  0 restores the local count. */
int splitlora_set_loss_normalizer(splitlora_ctx* ctx, int64_t n_valid_global);
/* on != 0: server_step stops after the backward pass (gradients in the server gradient buffer) and
 * leaves Eq. 4-5 to a later splitlora_server_update, after the caller has summed the gradients. */
int splitlora_set_deferred_server_update(splitlora_ctx* ctx, int on);
int splitlora_server_update(splitlora_ctx* ctx);
/* Device pointer and element count of an adapter arena: side SPLITLORA_SIDE_*, kind 0 = fp32
 * parameters, 1 = fp32 gradients.  Client arenas are [K, per-client]; the pointer stays valid while
 * the workspace is bound.  After writing parameters call splitlora_adapters_changed(side). */
int splitlora_adapter_buffer(splitlora_ctx* ctx, int side, int kind, float** dev, int64_t* count);
int splitlora_adapters_changed(splitlora_ctx* ctx, int side);
/* Eq. 8-9 with the clients spread over devices, in two halves around one sum over devices.
 * _local_sum: sum_{i local} (|D_i| / total_count) P_i for every client A and B, total_count = |D| over
 * ALL devices' clients; the result is left in a buffer of the workspace, *sum_dev (DEVICE pointer, HOST
 * out) with *count fp32 elements (one client's adapter set; the same on every device however many
 * clients each holds).  The caller adds these buffers up over devices in place (one all-reduce of
 * *count floats), then calls _broadcast, which writes the buffer to every local client (the downlink b3)
 * and, with per-client ranks, cuts each client back to its own rank afterwards.
 * sample_counts: HOST int64 [local clients].  Errors: SPLITLORA_ERR_COUNTS, SPLITLORA_ERR_WORKSPACE. */
int splitlora_aggregate_local_sum(splitlora_ctx* ctx, const int64_t* sample_counts, int64_t total_count,
                                  float** sum_dev, int64_t* count);
int splitlora_aggregate_broadcast(splitlora_ctx* ctx);

/* Device loss of the last server_step (fp32 scalar, DEVICE pointer into the workspace). */
int splitlora_loss_device(splitlora_ctx* ctx, const float** loss_dev);

const char* splitlora_last_error(const splitlora_ctx* ctx);
/* The stand-alone operators below that take no status word (attention, adapter gradients inside
 * lora_linear_bwd without a workspace word) record an expired bounded wait in a word the library keeps
 * per device.  This call synchronises the current device, copies that word to *code (HOST) and
 * returns SPLITLORA_ERR_TIMEOUT when it is non-zero, else SPLITLORA_OK.  The kernels of a context
 * report through splitlora_device_status instead. */
int splitlora_library_status(int32_t* code);
/* Reads the device status word (HOST out): 0, or the code left by a bounded wait that expired.
 * Synchronises the stream. */
int splitlora_device_status(splitlora_ctx* ctx, int32_t* code);
/* Number of kernels the context has launched since creation (HOST out). */
int splitlora_launch_count(const splitlora_ctx* ctx, int64_t* launches);
/* Per-kernel-class device time: when enabled, each launch is bracketed by CUDA events on the
 * context stream; splitlora_profile_report copies up to `cap` entries of {name, launches,
 * milliseconds} into HOST arrays and returns the number of classes in *n.
 * on: 0 off; 1 every launch class; 2 only the tensor-bound linear layers (classes "lora_linear_*",
 * "linear_*", "head_*"), which leaves two thirds of a round's launches without events between them. */
int splitlora_profile_enable(splitlora_ctx* ctx, int on);
int splitlora_profile_report(splitlora_ctx* ctx, char (*names)[48], int64_t* launches, double* ms,
                             int cap, int* n);

/* ---- stand-alone operators (kernel-level tests, the LoRA-linear sweep, bandwidth sweeps) ----
 * All pointers DEVICE; `stream` is a cudaStream_t.  `workspace` is scratch of at least the size
 * the matching *_workspace_bytes call reports. */

/* Grouped LoRA linear forward (Sec. II-C applied to G adapters over one shared frozen W):
 *   y[m,:] = x[m,:] W^T + bias + (alpha/r) (x[m,:] A_g^T) B_g^T,  g = m / (M/G)
 * x [M, in], W [out, in], bias [out] or NULL, y [M, out] in `dtype`; A [G, r, in], B [G, out, r] fp32.
 * M % G == 0; in bf16 mode M/G % 128 == 0, in % 64 == 0, out % 8 == 0. */
int splitlora_lora_linear_workspace_bytes(int dtype, int M, int n_in, int n_out, int r, int G, size_t* bytes);
int splitlora_lora_linear_fwd(int dtype, int use_tensor_cores, const void* x, const void* W, const void* bias,
                              const float* A, const float* B, float alpha, int M, int n_in, int n_out,
                              int r, int G, void* y, void* workspace, size_t workspace_bytes, void* stream);
/* Backward of the same layer (the G_A, G_B of Eq. 4-7 and the gradient passed on; W is frozen, no dW):
 *   dx = dy W + (alpha/r)(dy B_g) A_g ;  dA_g = (alpha/r)(dy_g B_g)^T x_g ;  dB_g = (alpha/r) dy_g^T (x_g A_g^T)
 * dy [M, out], dx [M, in] in `dtype`; dA [G, r, in], dB [G, out, r] fp32.  Wt is W transposed,
 * [in, out], in `dtype` (the caller keeps it; W is frozen so it is built once). */
int splitlora_lora_linear_bwd(int dtype, int use_tensor_cores, const void* x, const void* Wt, const void* dy,
                              const float* A, const float* B, float alpha, int M, int n_in, int n_out,
                              int r, int G, void* dx, float* dA, float* dB,
                              void* workspace, size_t workspace_bytes, void* stream);
/* The same forward in parts, so that they can be timed one by one: parts is a sum of 1 (the adapters'
 * compute copies and the rank-r projection h = x A_g^T, left in the workspace) and 2 (the product with
 * the frozen W with the rank-r term fused in; needs a preceding call with part 1 on the same workspace
 * and operands).  parts = 3 is splitlora_lora_linear_fwd. */
int splitlora_lora_linear_fwd_parts(int dtype, int use_tensor_cores, const void* x, const void* W, const void* bias,
                                    const float* A, const float* B, float alpha, int M, int n_in, int n_out,
                                    int r, int G, void* y, void* workspace, size_t workspace_bytes, void* stream,
                                    int parts);
/* The same backward in parts, so that they can be timed one by one: parts is a sum of 1 (the two rank-r
 * projections h = x A_g^T and dh = (alpha/r) dy B_g, which the other parts read from the workspace),
 * 2 (dx) and 4 (dA and dB).  Parts 2 and 4 need a preceding call with part 1 on the same workspace and
 * operands.  parts = 7 is splitlora_lora_linear_bwd. */
int splitlora_lora_linear_bwd_parts(int dtype, int use_tensor_cores, const void* x, const void* Wt, const void* dy,
                                    const float* A, const float* B, float alpha, int M, int n_in, int n_out,
                                    int r, int G, void* dx, float* dA, float* dB,
                                    void* workspace, size_t workspace_bytes, void* stream, int parts);
/* Frozen linear layer with a fused epilogue (the un-adapted projections of a block and their
 * backward products; W is frozen, so the backward is the same call on the transposed weight):
 *   epilogue 0: y = x W^T + bias                 1: z = x W^T + bias, y = gelu(z)
 *            2: y = x W^T + bias + r             3: y = (x W^T) * gelu'(r)
 * x [M, in], W [out, in], bias [out] or NULL, r / z / y [M, out], all in `dtype`.  status_word is a
 * zero-initialised device int that receives a code if a bounded wait inside the tensor-core kernel
 * expires (required when use_tensor_cores != 0 and dtype is bf16). */
int splitlora_linear(int dtype, int use_tensor_cores, const void* x, const void* W, const void* bias,
                     int epilogue, const void* r, void* z, int gelu_tanh, int M, int n_in, int n_out,
                     void* y, int* status_word, void* stream);
/* Compressed cut-layer hand-off.  The tensors that cross the cut (S in step a2 and dL/dS in step a4
 * of Sec. III-B) are what the paper's links carry; Sec. V (efficiency) names quantisation as the way
 * to shrink that exchange and fixes no format.  Format of this library: per token (row of d values)
 * one fp32 scale and d 8-bit E4M3 codes (4 exponent bits with bias 7, 3 mantissa bits, subnormals,
 * no infinities, largest finite value 448, code 0x7F / 0xFF = NaN, never produced):
 *   absmax = max |x[m,:]|, code[m,c] = E4M3(x[m,c] * (448 / absmax)), scales[m] = absmax / 448,
 * nearest value with ties to the even code, all in fp32; a row of zeros has scale 0 and codes 0.
 * _dequantize writes value(code[m,c]) * scales[m], rounded once to `dtype`.
 * x, y: device, [M, d] row-major in `dtype` (0 fp32, 1 bf16), 16-byte aligned; codes: device, [M, d]
 * bytes, 16-byte aligned; scales: device, [M] fp32; d a multiple of 8 (bf16) or 4 (fp32).  All
 * buffers are the caller's; nothing is allocated; work is enqueued on `stream`.  Bytes per token
 * handed off: d + 4 instead of 2 d (bf16) or 4 d (fp32).
 * Errors: SPLITLORA_ERR_ARG (null pointer, M < 1, d not a multiple of the vector width, dtype),
 * SPLITLORA_ERR_ALIGN, SPLITLORA_ERR_CUDA (launch failure). */
int splitlora_handoff_quantize(int dtype, const void* x, int64_t M, int d, uint8_t* codes, float* scales,
                               void* stream);
int splitlora_handoff_dequantize(int dtype, const uint8_t* codes, const float* scales, int64_t M, int d,
                                 void* y, void* stream);
/* out [cols, rows] = in [rows, cols]^T in `dtype` (for building Wt). */
int splitlora_transpose(int dtype, const void* in, int rows, int cols, void* out, void* stream);

/* Eq. 8-9 on raw buffers: params [K, P] fp32; weights HOST double [K] (already |D_i|/|D|);
 * every row is overwritten with sum_i w_i params[i, :].  P % 4 == 0. */
int splitlora_aggregate_buffers(float* params, int K, int64_t P, const double* weights, void* stream);

/* Causal multi-head attention on a fused qkv buffer [nseq*T, 3d] -> o [nseq*T, d], lse [nseq, H, T] fp32
 * (natural-log sum of exp of the scaled scores), and its backward -> dqkv [nseq*T, 3d]. */
int splitlora_attention_fwd(int dtype, int use_tensor_cores, const void* qkv, int nseq, int T, int n_head,
                            int d_model, void* o, float* lse, void* stream);
int splitlora_attention_bwd(int dtype, int use_tensor_cores, const void* qkv, const void* o, const float* lse,
                            const void* d_o, int nseq, int T, int n_head, int d_model, void* dqkv,
                            float* scratch_rowdot /* [nseq*T*H] */, void* stream);

/* Attention backward without caller scratch and without any allocation.  (The paper has no
 * counterpart; this serves callers that may not allocate device memory: code running under a
 * fixed memory budget handed out at start-up, or plug-ins inside a host application that owns the
 * allocator and forbids cudaMalloc after initialisation.)
 *
 * Same inputs, outputs and arithmetic as splitlora_attention_bwd, but the per-row scratch
 * (one float per sequence x head x position) lives in a fixed array inside the library: every
 * device that loads the library holds SPLITLORA_STATIC_ATTENTION_ROWS floats (4 MiB) until the
 * process exits.  Limits and rules:
 *   - nseq * T * n_head must not exceed SPLITLORA_STATIC_ATTENTION_ROWS, else the call returns
 *     SPLITLORA_ERR_TOO_LARGE and launches nothing;
 *   - the first call on a device looks up the array's device address (a cheap runtime query, no
 *     allocation); make that first call outside any stream capture;
 *   - all calls on a device share the one array, which keeps the previous call's contents; the
 *     call overwrites every element it later reads, so nothing needs clearing, but two calls that
 *     may overlap on the GPU (different streams) race on it: serialise them;
 *   - the call itself calls no cudaMalloc / cudaFree and no allocating library routine. */
#define SPLITLORA_STATIC_ATTENTION_ROWS (1 << 20)
#define SPLITLORA_ERR_TOO_LARGE -10   /* the problem does not fit a fixed-size internal buffer */
int splitlora_attention_bwd_static(int dtype, int use_tensor_cores, const void* qkv, const void* o,
                                   const float* lse, const void* d_o, int nseq, int T, int n_head,
                                   int d_model, void* dqkv, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPLITLORA_H_ */
