/*
 * treelstm.h - C ABI of the B200 (sm_100a) binary TreeLSTM library.
 *
 * The library evaluates a binary TreeLSTM over a forest (a batch of differently shaped binary
 * trees) by dependency-driven scheduling: every node whose children are finished is evaluated
 * together with all other ready nodes of the whole forest, forward and backward through the
 * tree structure.  Reference: "Improving the Expressiveness of Deep Learning Frameworks with
 * Recursion" (arXiv 1809.00832); the passages each call follows are cited at the call.
 *
 * Conventions
 *   - Every function returns an int: TREELSTM_OK (0) or a negative treelstm_status code.  No
 *     function throws, aborts or traps.
 *   - Unless a parameter is marked [host], array pointers are DEVICE pointers owned by the
 *     caller (e.g. PyTorch tensors); the library never frees them.  Scalars are passed by value.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All work
 *     of a call is enqueued on that stream.
 *   - Matrices are dense row-major, fp32, int32 indices.
 *   - A forest of n_nodes nodes is three int32 arrays: left[n], right[n] (both -1 for a leaf,
 *     both valid distinct node ids otherwise) and token[n] (vocabulary id of a leaf; ignored
 *     for internal nodes).  Node ids may be in any order (no topological numbering needed,
 *     Section 2.2); roots are the nodes that are nobody's child.
 *   - The cell (the paper writes it only as LSTM(...), Figures 1 and 2; this is the standard
 *     binary TreeLSTM):  in = [x ; h_l ; h_r],  z = W^T in + b  split into (i, f_l, f_r, o, u),
 *     c = sig(i)*tanh(u) + sig(f_l)*c_l + sig(f_r)*c_r,  h = sig(o)*tanh(c);  x = emb[token] and
 *     zero child state at a leaf, x = 0 at an internal node.
 */
#ifndef TREELSTM_H_
#define TREELSTM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define TREELSTM_API __attribute__((visibility("default")))
#else
#define TREELSTM_API
#endif

typedef struct treelstm treelstm_t;

typedef enum treelstm_status {
  TREELSTM_OK = 0,
  TREELSTM_ERR_INVALID_ARG = -1,        /* null pointer, non-positive size, workspace too small    */
  TREELSTM_ERR_INVALID_FOREST = -2,     /* child out of range, single child, two parents, cycle     */
  TREELSTM_ERR_TOKEN_OUT_OF_RANGE = -3, /* a leaf token outside [0, vocab)                          */
  TREELSTM_ERR_LABEL_OUT_OF_RANGE = -4, /* a label outside [0, C)                                   */
  TREELSTM_ERR_TIMEOUT = -5,            /* a bounded device-side wait expired                        */
  TREELSTM_ERR_CUDA = -6,               /* a CUDA runtime call failed; see treelstm_last_cuda_error */
  TREELSTM_ERR_NO_DEVICE = -7,          /* no sm_100 device is current                               */
  TREELSTM_ERR_UNSUPPORTED = -8,        /* size outside what the kernels support                     */
  TREELSTM_ERR_STATE = -9,              /* call order violated (e.g. backward without forward), or   */
                                        /* the current device is not the one the context was made on */
  TREELSTM_ERR_CHECK = -10              /* checked build only (-DTREELSTM_CHECKED): a kernel read an */
                                        /* index out of range from the schedule, or a state row was  */
                                        /* not written exactly as often as it must be                */
} treelstm_status;

/* precision of the gate contraction */
#define TREELSTM_FP32 0 /* fp32 operands, fp32 FMA accumulation, accurate activations            */
#define TREELSTM_BF16 1 /* x, h_l, h_r, W rounded to bf16; tcgen05 tensor cores, fp32 accumulate; */
                        /* bias, activations, c and the returned h stay fp32                      */

/* flags of treelstm_forward (or-ed together) */
#define TREELSTM_PER_LEVEL 0    /* one launch per wavefront; synchronises the stream once to read   */
                                /* the level table, returns device-detected errors directly          */
#define TREELSTM_PERSISTENT 1   /* one cooperative launch loops over the wavefronts with a bounded   */
                                /* grid-wide barrier; fully asynchronous (see treelstm_status_sync)  */
#define TREELSTM_SAVE_FOR_BACKWARD 2 /* keep every node's gate activations for treelstm_backward   */
#define TREELSTM_SUBFORESTS 4   /* bf16 only: the trees are dealt out to as many sub-forests as      */
                                /* thread-block clusters fit on the GPU; one cluster evaluates one   */
                                /* sub-forest wavefront by wavefront with its slice of the recurrent */
                                /* weights resident in shared memory and only the hardware cluster   */
                                /* barrier between wavefronts (trees are independent, Section 2.2).  */
                                /* One launch, asynchronous like TREELSTM_PERSISTENT, same results   */
                                /* and same reported schedule.  Where it does not apply (fp32, H     */
                                /* padded beyond 256, more than 24576 nodes) the call runs           */
                                /* TREELSTM_PERSISTENT instead; treelstm_last_mode tells which.      */

/* option keys of treelstm_set_option */
#define TREELSTM_OPT_SCHED_SINGLE_CTA_MAX 1 /* forests up to this many nodes are scheduled by one  */
                                            /* CTA in shared memory (0 forces the multi-CTA path)   */
#define TREELSTM_OPT_WAIT_LIMIT_CYCLES 2    /* upper bound of every device-side wait, in units of   */
                                            /* 1024 SM clock cycles                                  */
#define TREELSTM_OPT_MAX_CTAS 3             /* cap on the persistent grid (0 = all co-resident CTAs) */
#define TREELSTM_OPT_TIME_WAVEFRONT_KERNEL 4 /* 1: bracket the wavefront kernel launch(es) of each  */
                                            /* forward with CUDA events (treelstm_last_kernel_ms)    */
#define TREELSTM_OPT_TAIL_WIDTH 5           /* TREELSTM_PERSISTENT, bf16, H padded to <= 256: the last    */
                                            /* wavefronts of a forest, once every remaining one has at    */
                                            /* most this many nodes (default 32, largest value 64), may   */
                                            /* be finished by ONE thread-block cluster (a second launch): */
                                            /* recurrent weights resident in shared memory, states passed  */
                                            /* from child to caller through distributed shared memory.     */
                                            /* Decided by the library on the device (see below), same      */
                                            /* results bit for bit; 0 keeps every wavefront on the         */
                                            /* grid-wide kernel                                            */
#define TREELSTM_OPT_TAIL_MIN_LEVELS 6      /* 0 (default): the hand-over happens if a cost model fitted   */
                                            /* to cycle traces says that the narrow wavefronts save more   */
                                            /* than the second launch costs (deep, narrow forests: yes; a  */
                                            /* few narrow wavefronts on top of a wide forest: no).         */
                                            /* > 0: it happens whenever at least this many wavefronts      */
                                            /* remain                                                      */
#define TREELSTM_OPT_TAIL_MAX_NODES 7       /* forests with more nodes than this (default 4096) never      */
                                            /* launch the cluster kernel: the host knows the node count    */
                                            /* only, and a large forest has nothing to gain.  The second   */
                                            /* launch costs a few microseconds even when the cluster finds */
                                            /* nothing to do, so the library also leaves it out while the  */
                                            /* control block of the last forward it read back              */
                                            /* (treelstm_status_sync, treelstm_forward_host) said that the */
                                            /* forest had no tail worth handing over; the grid-wide kernel */
                                            /* keeps recording what the decision would have been, and the  */
                                            /* launch comes back with the first forest that has one        */
#define TREELSTM_OPT_OVERLAP_LAUNCH 8       /* 1 (default): the persistent wavefront kernel (bf16, fp32) is */
                                            /* launched as a programmatic dependent of the ready-set       */
                                            /* construction, so that its set-up (barriers, tensor memory,  */
                                            /* weights and biases asked into L2) runs while that kernel    */
                                            /* still works; it waits on the device for the schedule.  Such */
                                            /* a launch cannot be a cooperative one: that every CTA is     */
                                            /* resident then rests on the grid fitting the device (the     */
                                            /* library checks) and on the stream having the device to      */
                                            /* itself; otherwise the bounded grid barrier ends the call    */
                                            /* with TREELSTM_ERR_TIMEOUT.  0: cooperative launch in plain  */
                                            /* stream order (residency guaranteed by the runtime)          */
#define TREELSTM_OPT_LEAVES_FIRST_MIN_NODES 9 /* a kernel started that way evaluates the leaf wavefront    */
                                            /* before it waits for the schedule if the forest has at least */
                                            /* this many nodes (default 4096); smaller forests keep the    */
                                            /* order of work of the cooperative launch: their scheduler    */
                                            /* is too short to hide the two extra grid barriers            */
#define TREELSTM_OPT_DW_TENSOR_CORES 10     /* 1 (default): after a forward that kept its level table on   */
                                            /* the device, treelstm_backward forms dW, db and the input    */
                                            /* gradients of the leaves (dEmb_rows) in a second kernel on   */
                                            /* the tensor cores, every fp32 operand split into three bf16  */
                                            /* pieces (six products per term: fp32 accuracy); 0: fp32      */
                                            /* multiply-adds inside the one-launch backward                */

/*
 * treelstm_create - build a context for one set of parameters.
 *   Model: Section 2.2 (TreeLSTM cells composed in the shape of the input tree).
 *   H, E, vocab  hidden size, embedding size, vocabulary size (> 0).
 *   emb          [vocab][E]   embedding table.
 *   W            [E + 2H][5H] gate weights; rows [0,E) multiply x, [E,E+H) h_l, [E+H,E+2H) h_r;
 *                column blocks of width H in the order i, f_l, f_r, o, u.
 *   b            [5H]         gate bias, same column order.
 *   precision    TREELSTM_FP32 or TREELSTM_BF16.
 * The library copies (and for bf16 repacks, pads and converts) the parameters into device
 * memory it owns; the caller may free or change its arrays after the call returns (the call
 * synchronises `stream`).  *out is set to NULL on failure.  Release with treelstm_destroy.
 */
TREELSTM_API int treelstm_create(treelstm_t** out, int H, int E, int vocab, const float* emb, const float* W,
                    const float* b, int precision, void* stream);

/*
 * treelstm_create_recursive - a context for one of the paper's other two recursive models (Section
 * 6.1; Table 1 of Section 6.3 is measured on TreeRNN), evaluated by the same dependency-driven
 * schedule.  The paper prints neither cell; these are the published ones:
 *   TREELSTM_CELL_TREERNN   p   = tanh(W^T [h_l ; h_r] + b)
 *   TREELSTM_CELL_RNTN      p_j = tanh([h_l ; h_r]^T V_j [h_l ; h_r] + (W^T [h_l ; h_r])_j + b_j)
 * A leaf's state is its word vector, h = emb[token] (so the embedding width is H); there is no
 * cell state.
 *   emb [vocab][H], W [2H][H] (rows [0,H) multiply h_l, [H,2H) h_r), b [H],
 *   V [H][2H][2H] (one 2H x 2H slice per output unit; TREELSTM_CELL_RNTN only, else NULL).
 * fp32 arithmetic.  H <= 4096 (TreeRNN), H <= 128 (RNTN).  Parameters are copied (the tensor is
 * re-packed); the call synchronises `stream`.  Such a context takes treelstm_forward (flags
 * TREELSTM_PER_LEVEL or TREELSTM_PERSISTENT; c may be NULL and is not written), treelstm_roots
 * (root_c is not written), treelstm_forward_host (c, root_c not written), treelstm_status_sync,
 * treelstm_set_classifier, treelstm_backward_recursive (after a forward with
 * TREELSTM_SAVE_FOR_BACKWARD, which for these cells keeps nothing beyond h) and treelstm_destroy.
 */
#define TREELSTM_CELL_TREERNN 1
#define TREELSTM_CELL_RNTN 2
TREELSTM_API int treelstm_create_recursive(treelstm_t** out, int cell, int H, int vocab, const float* emb,
                                           const float* W, const float* b, const float* V, void* stream);

/* Re-read emb, W, b (same shapes as at create) after the caller changed them. Synchronises. */
TREELSTM_API int treelstm_update_weights(treelstm_t* ctx, const float* emb, const float* W, const float* b,
                            void* stream);

/*
 * treelstm_set_classifier - per-node softmax classifier used by treelstm_backward
 *   (Section 6.1: every node of every tree carries a label).
 *   Wc [H][C], bc [C]; copied; synchronises `stream`.  1 <= C <= 32.
 */
TREELSTM_API int treelstm_set_classifier(treelstm_t* ctx, int C, const float* Wc, const float* bc, void* stream);

TREELSTM_API int treelstm_set_option(treelstm_t* ctx, int key, long long value);

/*
 * treelstm_workspace_bytes - size of the caller-provided device scratch buffer that
 * treelstm_forward (and, if with_backward != 0, treelstm_backward) needs for forests of up to
 * max_nodes nodes.  Returns 0 on invalid arguments.  The buffer must be 256-byte aligned.
 */
TREELSTM_API size_t treelstm_workspace_bytes(const treelstm_t* ctx, int max_nodes, int with_backward);

/*
 * treelstm_forward - schedule the forest on the device and evaluate every node.
 *   Schedule: Section 4.1.1 (an operation is ready once all its inputs are resolved; completed
 *   operations release their dependants) and Section 4.1.2 (each invocation keeps a pointer to
 *   its caller).  Evaluation: Figure 2 (Section 3.1), all ready nodes of the forest at once;
 *   sibling subtrees are independent (Section 2.2).
 *   n_nodes       number of nodes (>= 0; 0 is a no-op that reports 0 levels).
 *   left,right,token  [n_nodes] the forest (see Conventions).
 *   h, c          [n_nodes][H] out: state of every node, indexed by node id.
 *   level         [n_nodes] out: wavefront of each node: 0 for a leaf, else
 *                 1 + max(level of its children).
 *   order         [n_nodes] out: node ids by ascending (level, node id) - the ready order.
 *   level_offset  [n_nodes + 2] out or NULL: wavefront l is order[level_offset[l] ..
 *                 level_offset[l+1]); entries past n_levels are unspecified.
 *   n_levels      [1] out (device): number of wavefronts.
 *   flags         TREELSTM_PER_LEVEL, TREELSTM_PERSISTENT or TREELSTM_SUBFORESTS, optionally
 *                 | TREELSTM_SAVE_FOR_BACKWARD.
 *   workspace     device scratch of at least treelstm_workspace_bytes(ctx, n_nodes, save) bytes;
 *                 with TREELSTM_SAVE_FOR_BACKWARD it must stay untouched until backward is done.
 * Errors: INVALID_ARG for bad arguments (nothing is launched).  A malformed forest or a token
 * out of range is detected on the device: no out-of-bounds access happens, the outputs are
 * unspecified, and the code is returned by this call (TREELSTM_PER_LEVEL) or by
 * treelstm_status_sync (TREELSTM_PERSISTENT, TREELSTM_SUBFORESTS).
 */
TREELSTM_API int treelstm_forward(treelstm_t* ctx, int n_nodes, const int32_t* left, const int32_t* right,
                     const int32_t* token, float* h, float* c, int32_t* level, int32_t* order,
                     int32_t* level_offset, int32_t* n_levels, int flags, void* workspace,
                     size_t workspace_bytes, void* stream);

/*
 * treelstm_status_sync - wait for the stream of the last forward/backward call and return the
 * status its kernels recorded (TREELSTM_OK, INVALID_FOREST, TOKEN/LABEL_OUT_OF_RANGE, TIMEOUT).
 */
TREELSTM_API int treelstm_status_sync(treelstm_t* ctx);

/*
 * treelstm_roots - after a forward on this context: the roots of the forest in ascending node
 * id, with their states gathered (Figure 2: root_state = TreeLSTM(root_idx)).
 *   root_ids [max_roots] out, root_h / root_c [max_roots][H] out (either may be NULL),
 *   n_roots [1] out (device).  Roots beyond max_roots are dropped.  Enqueued on `stream`.
 */
TREELSTM_API int treelstm_roots(treelstm_t* ctx, int max_roots, int32_t* root_ids, float* root_h, float* root_c,
                   int32_t* n_roots, void* stream);

/*
 * treelstm_backward - training step after treelstm_forward(... | TREELSTM_SAVE_FOR_BACKWARD) on
 * the same context: mean softmax cross-entropy of the classifier on every node's h, and
 * backpropagation through structure.
 *   Section 4.2.2: the gradient computation recurses at the same positions as the forward
 *   computation (here: wavefronts in reverse, parents before children); Sections 4.2.1 and 5:
 *   each node instance uses its own retained forward values (here: dense per-node arrays, the
 *   node id being the unique key).
 *   labels       [n_nodes] class of every node, in [0, C).
 *   loss         [1] out (device): mean over all nodes of -log softmax(Wc^T h_n + bc)[label_n].
 *   dW [E+2H][5H], db [5H], dWc [H][C], dbc [C]  out: gradients (overwritten, not accumulated).
 *   touched_ids  [n_leaves] out: sorted unique leaf tokens; dEmb_rows [n_leaves][E] out: one
 *                summed gradient row per touched id (duplicates accumulate); n_touched [1] out.
 *                Rows past n_touched are unspecified.
 * The forest arrays, h, c, order, level and the workspace of the forward call must still be
 * valid and unchanged.  After a TREELSTM_PERSISTENT or TREELSTM_SUBFORESTS forward the loss and all
 * wavefronts are one cooperative launch that reads the level table on the device (asynchronous, no
 * host round trip; a label out of range is reported by treelstm_status_sync), followed - unless
 * TREELSTM_OPT_DW_TENSOR_CORES is 0 - by one tensor-core launch for dW, db and dEmb_rows (their sums
 * run over all nodes and depend on no wavefront order); after a TREELSTM_PER_LEVEL forward it is one
 * launch pair per wavefront, driven by the level table the forward already read back.  Computes at
 * fp32 accuracy from the fp32 parameters whatever the forward precision.
 */
TREELSTM_API int treelstm_backward(treelstm_t* ctx, const int32_t* labels, float* loss, float* dW, float* db,
                      float* dWc, float* dbc, int32_t* touched_ids, float* dEmb_rows,
                      int32_t* n_touched, void* stream);

/*
 * treelstm_backward_recursive - the same training step for a context made by
 * treelstm_create_recursive (TreeRNN or RNTN, Section 6.1), after treelstm_forward(... |
 * TREELSTM_SAVE_FOR_BACKWARD) on it; treelstm_set_classifier works on such a context as on any other.
 *   An internal node n with x = [h_l ; h_r] and h_n = tanh(z_n):  dz = dh_n * (1 - h_n^2);
 *   dW += x (x) dz;  db += dz;  RNTN: dV_j += dz_j * x (x) x;  the children's dh receive
 *   W dz (+ RNTN: sum_j dz_j (V_j + V_j^T) x);  a leaf's state is its word vector, so its dh is
 *   added to the gradient row of its token.  Wavefronts in reverse (Section 4.2.2).
 *   labels, loss, dWc [H][C], dbc [C], touched_ids, n_touched: as for treelstm_backward.
 *   dW [2H][H], db [H]  out;  dV [H][2H][2H] out (RNTN; may be NULL for TreeRNN);
 *   dEmb_rows [n_leaves][H] out: one summed row per touched id.
 * All device pointers; gradients are overwritten.  The level table is read back once (the call
 * synchronises the stream of the forward if that was a TREELSTM_PERSISTENT one), then one launch per
 * phase and wavefront; fp32.  Errors: as treelstm_backward; TREELSTM_ERR_STATE on a TreeLSTM context
 * (and treelstm_backward returns it on a TreeRNN / RNTN context).
 */
TREELSTM_API int treelstm_backward_recursive(treelstm_t* ctx, const int32_t* labels, float* loss, float* dW,
                                             float* db, float* dV, float* dWc, float* dbc, int32_t* touched_ids,
                                             float* dEmb_rows, int32_t* n_touched, void* stream);

/*
 * treelstm_forward_host - the same forward for callers whose data lives in HOST memory: copies
 * the forest to the device, runs treelstm_forward with `flags`, copies the requested results
 * back and synchronises.  Device staging and workspace come from the buffer given with
 * treelstm_set_host_staging; without one they are owned by the context and grown on demand
 * (cudaMalloc on the first call or when n_nodes grows).
 *   left,right,token [host][n_nodes] in (pinned memory makes the copies asynchronous).
 *   h, c           [host][n_nodes][H] out, or NULL to skip the all-node states.
 *   level, order   [host][n_nodes] out, or NULL.
 *   max_roots, root_ids [host][max_roots], root_h, root_c [host][max_roots][H]: the roots in
 *                  ascending node id with their states, or NULL; n_roots [host][1] out or NULL.
 *   n_levels       [host][1] out or NULL.
 * Copies are few and small, so their number matters: if right == left + n_nodes and token == right +
 * n_nodes the forest goes up in one copy, and if root_h == (float*)(root_ids + max_roots) and
 * root_c == root_h + max_roots * H (with max_roots <= n_nodes) the roots come back in one.
 * Returns the device status as well (it has synchronised).
 */
TREELSTM_API int treelstm_forward_host(treelstm_t* ctx, int n_nodes, const int32_t* left, const int32_t* right,
                          const int32_t* token, float* h, float* c, int32_t* level, int32_t* order,
                          int32_t* n_levels, int max_roots, int32_t* root_ids, float* root_h,
                          float* root_c, int32_t* n_roots, int flags, void* stream);

/*
 * treelstm_host_staging_bytes / treelstm_set_host_staging - let the caller own the device memory
 * treelstm_forward_host stages through (forest arrays, schedule, all-node states, root pack,
 * workspace), so that the library allocates nothing on that path either.  (Plumbing; the paper has
 * no counterpart.)
 *   treelstm_host_staging_bytes: bytes needed for forests of up to max_nodes nodes (0 on invalid
 *   arguments).
 *   treelstm_set_host_staging: device_buffer is 256-byte aligned device memory of `bytes` bytes that
 *   stays valid until it is replaced, withdrawn (device_buffer = NULL: the library goes back to its
 *   own buffers) or the context is destroyed; the library never frees it.  A later
 *   treelstm_forward_host whose forest needs more than `bytes` returns TREELSTM_ERR_INVALID_ARG and
 *   launches nothing.
 */
TREELSTM_API size_t treelstm_host_staging_bytes(const treelstm_t* ctx, int max_nodes);
TREELSTM_API int treelstm_set_host_staging(treelstm_t* ctx, void* device_buffer, size_t bytes);

/*
 * treelstm_schedule_static - the ready-set construction of treelstm_forward on its own, for
 * callers that are not allowed to allocate device memory.  (The paper has no counterpart to this
 * call; it exists for the sake of such callers only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a framework that owns all
 * device memory through its own pool and forbids side allocations, in a process whose memory
 * budget was fixed at start-up, or on a latency-critical path where an allocation (which may
 * synchronise the whole device) is unacceptable.  Such a caller cannot create a context
 * (treelstm_create copies the parameters into memory it allocates) and has nowhere to get the
 * workspace treelstm_forward wants.  This call needs neither: it takes no context, and the
 * scratch the scheduling kernel needs (caller links, sort buffers, control block - about 193 KB)
 * lives in a fixed array inside the library's device image, present on every GPU that loads the
 * library until the process exits.
 *
 *   n_nodes       0 .. TREELSTM_STATIC_MAX_NODES (16384); more returns TREELSTM_ERR_UNSUPPORTED
 *                 and launches nothing.
 *   left,right,token  [n_nodes] the forest, as for treelstm_forward; vocab bounds the leaf tokens.
 *   level, order  [n_nodes] out;  level_offset [n_nodes + 2] out;  n_levels [1] out - the same
 *                 values treelstm_forward reports.
 *   status        [1] out (device): TREELSTM_OK, TREELSTM_ERR_INVALID_FOREST or
 *                 TREELSTM_ERR_TOKEN_OUT_OF_RANGE as found by the kernel; read it after the stream
 *                 has finished.  On an error the other outputs are unspecified.
 * The call only enqueues work on `stream` (one kernel and one 4-byte copy of the status word; for
 * the empty forest three small memory sets and that copy); it never calls cudaMalloc, cudaFree or
 * any routine that allocates.  The first call on each device looks
 * up the device address of the built-in scratch array (with that device current); make that first
 * call outside any stream capture.  All calls on a device share the one scratch array, and it keeps
 * whatever the previous call left there - the call clears the parts that must start from zero
 * itself - so two calls whose work overlaps on the GPU (different streams without ordering between
 * them) corrupt each other: order them.
 */
#define TREELSTM_STATIC_MAX_NODES 16384
TREELSTM_API int treelstm_schedule_static(int n_nodes, const int32_t* left, const int32_t* right,
                                          const int32_t* token, int vocab, int32_t* level, int32_t* order,
                                          int32_t* level_offset, int32_t* n_levels, int32_t* status,
                                          void* stream);

/*
 * treelstm_last_kernel_ms - device time of the wavefront kernel launch(es) of the last forward
 * (the persistent kernel, or the per-level launches together), measured with CUDA events on the
 * call's stream.  Needs TREELSTM_OPT_TIME_WAVEFRONT_KERNEL = 1 before that forward; waits for the
 * kernel to finish.  ms [host][1] out.
 */
TREELSTM_API int treelstm_last_kernel_ms(treelstm_t* ctx, float* ms);

/*
 * treelstm_selftest_waits - exercises the bounded device-side waits without any fault: one CTA
 * waits on a shared-memory barrier nobody arrives at, then on a grid barrier that expects a CTA
 * that does not exist.  Both must give up after the limit set with TREELSTM_OPT_WAIT_LIMIT_CYCLES
 * (set a small one first) and record TREELSTM_ERR_TIMEOUT; the context stays usable.  (Robustness
 * aid; the paper has no counterpart.)
 *   workspace  device scratch, >= 256 bytes, 256-byte aligned (its first 256 bytes are overwritten).
 *   result     [4] out (device): {first wait succeeded (must be 0), status after it (must be
 *              TREELSTM_ERR_TIMEOUT), second wait succeeded (0), status after it (TIMEOUT)}.
 * Asynchronous on `stream`.
 */
TREELSTM_API int treelstm_selftest_waits(treelstm_t* ctx, void* workspace, size_t workspace_bytes,
                                         int32_t* result, void* stream);

/* Number of kernels the last forward / backward call on this context launched. */
TREELSTM_API int treelstm_last_launch_count(const treelstm_t* ctx);

/* Which evaluation the last successful forward ran: TREELSTM_PER_LEVEL, TREELSTM_PERSISTENT or
 * TREELSTM_SUBFORESTS; -1 before any forward. */
TREELSTM_API int treelstm_last_mode(const treelstm_t* ctx);

/* Number of sub-forests TREELSTM_SUBFORESTS splits a forest into on this context's device (the
 * number of co-resident clusters); 0 if that mode is not available for this context. */
TREELSTM_API int treelstm_subforest_count(const treelstm_t* ctx);

/*
 * treelstm_tile_plan - how the bf16 wavefront kernel would cut a wavefront of `rows` ready nodes into
 * tiles on a grid of n_ctas CTAs (the kernel takes the same decision on the device for every
 * wavefront; this host-side view exists for tests and tuning; the paper has no counterpart).
 *   out [host][10]: rows per tile (32 / 64 / 128), unit groups of 8 hidden units per tile (1 / 2 /
 *   4), number of tiles, first tile of the split last round (= number of fat tiles if it is not
 *   split), log2 of the number of pieces a fat tile of that round is cut into, K blocks per operand
 *   box, boxes per tile, ring stages, bytes per stage, bytes of the ring.
 * No CUDA call is made.
 */
TREELSTM_API int treelstm_tile_plan(int rows, int H, int E, int n_ctas, int leaf, int32_t* out);

/* cudaError_t of the last failed CUDA call on this context (0 if none). */
TREELSTM_API int treelstm_last_cuda_error(const treelstm_t* ctx);

/* Frees everything the context owns.  NULL is allowed. */
TREELSTM_API int treelstm_destroy(treelstm_t* ctx);

/* Static description of a status code. */
TREELSTM_API const char* treelstm_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* TREELSTM_H_ */
