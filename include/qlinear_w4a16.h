/*
 * qlinear_w4a16 - weight-only int4, group-quantised linear layers for the verify step of
 * speculative decoding, for NVIDIA B200 (sm_100a).
 *
 *     Y[M,N] = X[M,K] * W[K,N],     W[k,n] = (q[k,n] - z[k/g,n]) * s[k/g,n]
 *
 * q: int4 codes, s: bf16 per-group scales, z: int4 per-group zero points, X and Y: bf16,
 * M = 1..64 drafted tokens, accumulation in fp32.
 *
 * Where this comes from.  The paper's quantised target keeps every linear layer as INT4 codes W_q
 * under frozen per-group scales s; its weights are the element-wise product of s and W_q
 * (Section 2.1), in groups of 128 along K with symmetric codes (Section 3.3; symmetric means
 * z == 8 here), and it is served with 16-bit activations (W4A16, Section 2.1).  The drafter
 * proposes blocks of 16 tokens (Section 3.2) that the target scores in one forward pass
 * (Section 2.2), so each projection runs with M = 16 rows per verify step, and the greedy token
 * of every row must be exactly the one the quantised layer defines, because verification does not
 * change the output (Section 4).  The paper describes no kernel; packing order, zero points and
 * shapes are fixed by this header.
 *
 * Conventions for every entry point
 *  - Pointers are DEVICE pointers unless a parameter says HOST.  The caller allocates and owns
 *    every buffer; the library allocates nothing and never frees.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only
 *    enqueue work on it and return a host-side status at once; no call synchronises unless it
 *    says so.
 *  - Return value: a ql_status.  Anything but QL_OK means that nothing was launched (argument
 *    errors) or that a CUDA call failed (QL_ERR_CUDA).  A wrong result is never returned
 *    silently for an unsupported shape.
 *  - Supported shapes: 1 <= M <= 64, g in {64, 128}, K % g == 0, N % 128 == 0, K, N > 0.
 *    X, Y, scale, wq: 16-byte aligned; leading dimensions multiples of 8 elements.
 *  - Results are bit-identical from run to run for identical inputs, shapes and device
 *    (all reductions are in a fixed order; no floating-point atomics).
 *  - NaN / Inf in X or the scales are not checked and propagate.
 *  - There is no CPU fallback and no other backend: without a B200-class device the compute
 *    entry points return QL_ERR_CUDA / QL_ERR_UNSUPPORTED.
 */
#ifndef QLINEAR_W4A16_H_
#define QLINEAR_W4A16_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QL_OK = 0,
  QL_ERR_NULL = 1,           /* a required pointer is NULL */
  QL_ERR_SHAPE = 2,          /* M, K, N, g or a leading dimension outside the supported set */
  QL_ERR_ALIGN = 3,          /* a pointer or leading dimension is not aligned as required */
  QL_ERR_UNSUPPORTED = 4,    /* path not available for this shape / device */
  QL_ERR_WORKSPACE = 5,      /* packed buffer or workspace too small */
  QL_ERR_CUDA = 6,           /* a CUDA runtime call failed (launch, copy, attribute) */
  QL_ERR_DEVICE_TIMEOUT = 7  /* a bounded wait inside a kernel ran out (read via ql_device_status) */
} ql_status;

/* Compute paths of qlinear_w4a16 (what ql_select_path returns, what qlinear_w4a16_path takes). */
typedef enum {
  QL_PATH_AUTO = 0,
  QL_PATH_MMA = 2,   /* warp-level bf16 tensor-core MMA (mma.sync), registers-resident operands */
  QL_PATH_TC5 = 3    /* tcgen05 bf16 MMA, weights written to tensor memory, accumulators in TMEM */
} ql_path;            /* (1 is not used: a CUDA-core path would need M FMAs per weight and was not built) */

const char* ql_status_str(int status);

/* Bytes of the packed weight buffer for a [K,N] matrix with group size g:
 * (N/128)*(K/g)*(64*g + 320) - codes, bf16 scales and 4-bit zero points, no padding.
 * Returns 0 for an unsupported (K, N, g). */
size_t ql_packed_bytes(int K, int N, int g);

/* Bytes of workspace that qlinear_w4a16 / qlinear_stack_w4a16 need for any call with
 * M <= M_max and N <= N_max (split-K partial tiles, tile counters, arg-max candidates, a status
 * word).  Returns 0 for unsupported arguments.  Needs no device. */
size_t ql_workspace_bytes(int M_max, int N_max);

/* Initialises a workspace (asynchronously, on `stream`): zero everywhere, except for the region
 * through which thread blocks of qlinear_stack_w4a16 hand partial rows to one another, which is
 * filled with the bit pattern that means "nothing waiting" (all ones).  Call once after allocating
 * the workspace, after the memory was used for anything else (the attention call included), and
 * again after a call reported QL_ERR_DEVICE_TIMEOUT (until then the status word stays set, and
 * qlinear_stack_w4a16 launches on that workspace run through without waiting for anything: their
 * results are not valid, and ql_device_status keeps saying why).  The kernels leave the control words zeroed
 * and that region empty when they finish, so no further initialisation is needed between calls.  One
 * workspace serves one stream at a time: calls that may overlap on the GPU need separate
 * workspaces. */
int ql_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Reads the workspace's status word into *host_out (QL_OK or QL_ERR_DEVICE_TIMEOUT).
 * SYNCHRONISES `stream`.  host_out is a HOST pointer. */
int ql_device_status(const void* workspace, int* host_out, void* stream);

/* Same, but returns the whole status word: bits 0-7 the ql_status, bits 8-15 an identifier of the
 * wait that gave up, bits 16-31 the index of the thread block it happened in (diagnostics). */
int ql_device_status_raw(const void* workspace, int* host_out, void* stream);

/*
 * qpack_w4_g128 - repack a quantised weight matrix into the tile layout the GEMM kernels stream.
 * (Input: the checkpoint-side representation of Section 2.1's W_q and s; output: opaque.)
 *
 *   wq     [K/8, N] uint32 row-major; word (r, n) holds the codes of rows k = 8r+j of column n at
 *          bits [4j, 4j+4)  (8 codes per word along K, low nibble first)
 *   scale  [K/g, N] bf16 bit patterns
 *   zero   [K/g, N] one code 0..15 per byte; NULL = symmetric weights, z == 8 everywhere
 *   g      64 or 128 (the name keeps the paper's group size; g is a parameter)
 *   packed out, ql_packed_bytes(K,N,g) bytes, 16-byte aligned
 *
 * Layout written (T = n / 128, G = k / g): chunk (T, G) starts at byte (T*(K/g)+G)*(64g+320) and
 * holds  [0,64g): 32-bit words number (c*128 + n%128)*4 + j, the 8 codes of column n, rows
 * g*G + 32c + 8j + i (i = 0..7), code i in nibble (i>>1) + 4*(i&1);  [64g, 64g+256): the 128
 * bf16 scales of (G, 128T..128T+127);  [64g+256, 64g+320): their 128 zero points, 4 bits each,
 * word n%128 >> 3, nibble n & 7.   Pure integer permutation: the result is fully determined.
 * Errors: QL_ERR_NULL, QL_ERR_SHAPE, QL_ERR_ALIGN, QL_ERR_WORKSPACE (packed_bytes too small).
 */
int qpack_w4_g128(const uint32_t* wq, const uint16_t* scale, const uint8_t* zero,
                  int K, int N, int g, void* packed, size_t packed_bytes, void* stream);

/*
 * qrequant_pack_w4 - grid-preserving re-quantisation, fused with the repack (Section 2.1: after
 * distillation the updated BF16 weights are rounded back onto the same quantisation grid, which
 * gives new INT4 codes under the original, frozen scales).
 *
 *   w       [K, N] bf16 bit patterns, row-major: the updated weights
 *   scale   [K/g, N] bf16, zero [K/g, N] or NULL (z == 8): the frozen grid, as in qpack_w4_g128
 *   packed  out, ql_packed_bytes(K,N,g) bytes: the layout of qpack_w4_g128, holding the codes
 *           clamp( rne( float32(w) / float32(scale) ) + zero, 0, 15 )
 * The quotient is the IEEE float32 division, rne rounds halves to the even integer: the result
 * is fully determined (bit-exact against the reference).  Errors as qpack_w4_g128.
 */
int qrequant_pack_w4(const uint16_t* w, const uint16_t* scale, const uint8_t* zero,
                     int K, int N, int g, void* packed, size_t packed_bytes, void* stream);

/*
 * qlinear_w4a16 - Y = X * dequant(packed)  (Section 2.1's s (.) W_q applied to a block of M
 * drafted tokens, Section 2.2), optionally followed by the greedy token of each row (Section 4).
 *
 *   packed      output of qpack_w4_g128 for the same (K, N, g)
 *   X           [M, K] bf16, row-major, leading dimension K
 *   Y           [M, N] bf16, row-major, leading dimension N; round-to-nearest-even of the fp32
 *               accumulator.  May be NULL if only argmax_out is wanted.
 *   argmax_out  [M] int32 or NULL: index of the largest fp32 accumulator of each row (taken
 *               before rounding to bf16), lowest index on ties
 *   workspace   >= ql_workspace_bytes(M, N) bytes, initialised by ql_workspace_init
 *
 * Weights enter the tensor core as the exact integers q - z; the per-group scale multiplies the
 * fp32 group sum.  The path (MMA / TC5) is chosen from (M, K, N, g); see ql_select_path.
 * Errors: QL_ERR_NULL, QL_ERR_SHAPE, QL_ERR_ALIGN, QL_ERR_WORKSPACE, QL_ERR_CUDA.
 */
int qlinear_w4a16(const void* packed, const uint16_t* X, uint16_t* Y, int32_t* argmax_out,
                  int M, int K, int N, int g,
                  void* workspace, size_t workspace_bytes, void* stream);

/* Same as qlinear_w4a16 with the compute path forced (benchmarks and tests).
 * QL_ERR_UNSUPPORTED if that path cannot run the shape. */
int qlinear_w4a16_path(const void* packed, const uint16_t* X, uint16_t* Y, int32_t* argmax_out,
                       int M, int K, int N, int g,
                       void* workspace, size_t workspace_bytes, void* stream, int path);

/* The path qlinear_w4a16 takes for a shape (a ql_path other than AUTO), or a negative ql_status. */
int ql_select_path(int M, int K, int N, int g);

/* How a linear launched on its own would be set up, without launching (needs no device: it then
 * plans for 148 SMs).  out (HOST, 4 ints): [0] the path taken (path == QL_PATH_AUTO: the selected
 * one), and for the warp-level MMA path [1] the depth of the shared-memory ring, [2] the groups of
 * X held in shared memory per thread block, [3] 0 if the X columns a block needs stay resident,
 * else the number of chunks after which they are reloaded (large M with long K).
 * Errors: QL_ERR_NULL, QL_ERR_SHAPE, QL_ERR_UNSUPPORTED. */
int ql_linear_plan(int M, int K, int N, int g, int path, int out[4]);

/*
 * qlinear_stack_w4a16 - run a list of operations in order on one stream: the projections of one
 * or many decoder layers (q/k/v/o, gate/up/down) and the LM head of one verify step (Section 2.2:
 * the target's forward pass over a drafted block), with the element-wise glue that chains them
 * in the benchmark stack.  `ops` is a HOST array, read before the call returns.
 *
 *   QL_OP_LINEAR             out[M,N] = in0[M,K] * dequant(packed);  argmax_out optional
 *   QL_OP_UNIT_RMS           out[m,:] = bf16( in0[m,:N] / sqrt(mean_n in0[m,n]^2) )      (fp32 math)
 *   QL_OP_SILU_MUL_UNIT_RMS  a = silu(in0) * in1 (fp32);  out[m,:] = bf16( a / sqrt(mean a^2) )
 *
 * Verification tail (Section 2.2: the target keeps the longest prefix of the drafted block that it
 * agrees with; Section 4: under greedy decoding the output is unchanged): a LINEAR with argmax_out
 * may also be given draft_ids[M] and accept_out[2].  The kernel then compares, on the device and
 * without a host round trip, the greedy token of row i with draft_ids[i], i = 0..M-1, and writes
 * accept_out[0] = a, the number of leading rows that agree, and accept_out[1] = the greedy token of
 * row a (the target's own token at the first disagreement), or -1 if all M rows agree.  Which row
 * confirms which drafted token is the caller's choice (it builds draft_ids; an entry of -1 never
 * agrees).  M <= 16 only (QL_ERR_UNSUPPORTED otherwise).
 *
 * in0/in1/out are bf16 with leading dimensions ld_in (in0 and in1) and ld_out, so an operation
 * can read a column slice of a wider tensor.  Operation i sees the results of operations < i.
 * The packed weights of every LINEAR must be complete before the call and must not change while
 * it runs: a linear may start streaming its weights while the operation before it finishes.
 * Runs of operations with M <= 16 and one group size execute as ONE cooperative launch of a
 * persistent kernel.  A list that consists of pairwise independent plain linears with one common
 * M above 16 does too: every linear is cut into slabs of 16 rows, which join the one stream of
 * chunks (the weights are unpacked once per slab).  Other operations with M > 16 are launched
 * one by one.  A run of plain linears no two of which share a buffer (other than inputs
 * both only read) is treated as one long stream of chunks cut into one contiguous piece per
 * thread block (the X operand stays in shared memory per operation where it fits and follows the
 * chunks through a ring of slots where it does not); any other run is a chain - glue folded into the
 * neighbouring linears, gate/up pairs fused, every operation waiting for the one before it.  The
 * thread blocks wait for one another with bounded waits, so a stream that is starved of SMs for
 * more than 2 s reports QL_ERR_DEVICE_TIMEOUT in the status word instead of hanging.
 * ql_stack_plan tells what a list turns into.  The call stages the fused
 * operation descriptors from host memory into the workspace with an asynchronous copy, so it is
 * not meant to be recorded by stream capture.
 * A call that resolves to one launch of the persistent kernel is remembered per host thread: the
 * same call again (byte-identical operation list, same workspace, size and stream, and nothing
 * staged into any workspace by any thread in between) skips planning and the descriptor copy and
 * only launches.  A changed field of an operation, another list, ql_workspace_init, a
 * qattn_swa_bf16 call or any ql_debug_* setter makes the next call plan again.  (The workspace
 * belongs to the library between calls: a caller that writes into it must call ql_workspace_init.)
 * Errors: as qlinear_w4a16, reported for the first offending operation; nothing is launched
 * unless every operation validates.
 */
typedef enum { QL_OP_LINEAR = 0, QL_OP_UNIT_RMS = 1, QL_OP_SILU_MUL_UNIT_RMS = 2 } ql_op_kind;

typedef struct ql_op {
  int32_t kind;          /* ql_op_kind */
  int32_t M;             /* rows, 1..64 */
  int32_t K;             /* LINEAR: contraction length; glue: ignored */
  int32_t N;             /* LINEAR: output columns; glue: columns processed */
  int32_t g;             /* LINEAR: group size; glue: ignored */
  int32_t ld_in;         /* leading dimension of in0 / in1, elements */
  int32_t ld_out;        /* leading dimension of out, elements */
  int32_t reserved;      /* must be 0 */
  const void* packed;    /* LINEAR: packed weights */
  const uint16_t* in0;   /* bf16 */
  const uint16_t* in1;   /* SILU_MUL_UNIT_RMS: second operand */
  uint16_t* out;         /* bf16; LINEAR: may be NULL when argmax_out is given */
  int32_t* argmax_out;   /* LINEAR: [M] or NULL */
  const int32_t* draft_ids;  /* LINEAR with argmax_out: [M] drafted tokens to verify, or NULL */
  int32_t* accept_out;       /* with draft_ids: [2] accepted-prefix length, bonus token */
} ql_op;

int qlinear_stack_w4a16(const ql_op* ops, int n_ops,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * ql_stack_plan - what qlinear_stack_w4a16 would do with an operation list, without launching
 * anything (needs no device: it then plans for 148 SMs).  Same validation and errors.
 * counts (HOST, 8 ints): [0] launches of the persistent stack kernel, [1] fused operations inside
 * them, [2] of which gate/up pairs run as one dual operation, [3] glue operations folded into their
 * neighbouring linears, [4] fused operations that do not wait for their predecessor, [5] linears
 * launched on their own, [6] glue operations launched on their own, [7] of the launches in [0],
 * those whose operations are pairwise independent plain linears and run as one stream of chunks.
 */
int ql_stack_plan(const ql_op* ops, int n_ops, void* workspace, size_t workspace_bytes, int counts[8]);

/*
 * qlinear_stack_w4a16_host - the same step for a caller whose activations live in HOST memory:
 * copies host_in (in_bytes) to dev_in, runs the stack, copies out_bytes from dev_out to host_out,
 * then SYNCHRONISES `stream`.  host_in / host_out are HOST pointers (pinned memory makes the
 * copies asynchronous up to the final synchronisation); dev_in / dev_out are device buffers that
 * operations of the stack read and write.  Either copy is skipped when its byte count is 0.
 */
int qlinear_stack_w4a16_host(const ql_op* ops, int n_ops,
                             const void* host_in, void* dev_in, size_t in_bytes,
                             const void* dev_out, void* host_out, size_t out_bytes,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * qlinear_w4a16_static - qlinear_w4a16 for callers that cannot hand over a workspace.
 * (No counterpart in the paper: this entry point exists for the sake of its callers only.)
 *
 * Who needs it: code that runs where device memory cannot be obtained - a plugin or a callback
 * inside somebody else's engine that owns the allocator, a real-time loop that may not call the
 * allocator after start-up, a process whose memory budget was handed out before this library was
 * loaded.  Such a caller has its inputs and outputs, but nowhere to put the kernel's scratch
 * (split-K partial tiles, tile counters, arg-max candidates, status word).  Here that scratch is
 * a static device array inside the library, about 5.8 MB, which every GPU that loads the library
 * holds until the process exits.  The call allocates nothing and calls nothing that allocates.
 *
 *   arguments as qlinear_w4a16, without the workspace; leading dimensions are K and N
 *   limits: M <= 16 and N <= 16384 (QL_ERR_WORKSPACE beyond them); K, g as qlinear_w4a16
 *
 * The first call on a device looks up the array's device address (once per device, with that
 * device current); make that first call outside any stream capture.  Every call shares the one
 * array, which keeps the contents of the call before: the control words are cleared on the stream
 * at the start of each call, everything else is written before it is read.  Two calls that may
 * overlap on the GPU (different streams) race on the array - serialise them.
 * The result is the one of qlinear_w4a16_path(..., QL_PATH_MMA) for the same arguments.
 * ql_static_status reads the array's status word (QL_OK or QL_ERR_DEVICE_TIMEOUT) and
 * SYNCHRONISES the stream; host_out is a HOST pointer.
 */
int qlinear_w4a16_static(const void* packed, const uint16_t* X, uint16_t* Y, int32_t* argmax_out,
                         int M, int K, int N, int g, void* stream);
int ql_static_status(int* host_out, void* stream);

/* Symmetric sliding-window attention of a drafted block (paper Section 3.3, "Drafter SWA": the
 * drafter's mask-token queries attend bidirectionally, each restricted to a fixed-size window that
 * is symmetric around the query; the window is applied inside the attention computation only, the
 * key/value cache stays complete; sequences that fit into the window are attended in full.
 * Section 2.3 for why the drafter has it).
 *
 *   query i (0 <= i < n_q) stands at position p0 + i and sees the keys k with
 *   |k - (p0 + i)| <= window / 2 (integer division), clipped to [0, T); every key if T <= window.
 *   out[i, h, :] = sum_k softmax_k(Q[i,h,:] . K[k, h / (Hq/Hkv), :] / sqrt(d)) * V[k, h / (Hq/Hkv), :]
 *   over the visible keys; bf16 in and out, fp32 arithmetic (probabilities enter the second
 *   contraction with 16 significant bits).
 *
 *   Q    DEVICE, bf16 [n_q][Hq][d], ld_q elements between consecutive queries (>= Hq*d)
 *   K, V DEVICE, bf16 [T][Hkv][d], ld_kv elements between consecutive positions (>= Hkv*d):
 *        the complete cache; positional rotation, if any, has been applied before
 *   out  DEVICE, bf16 [n_q][Hq][d], ld_out elements between consecutive queries
 *   1 <= n_q <= 16, d == 128, Hq/Hkv in {1, 2, 4, 8}, 0 <= p0, p0 + n_q <= T, window >= 0;
 *   leading dimensions multiples of 8, pointers 16-byte aligned
 *   workspace DEVICE, >= ql_attn_workspace_bytes(Hq, Hkv) bytes, zeroed once with ql_workspace_init
 *        (it is NOT the workspace of the linear calls: the two may not share memory that is in use
 *        at the same time); holds the partial rows of the key pieces and one counter per head;
 *        calls that may overlap on the GPU (different streams) need workspaces of their own
 *
 * Asynchronous on `stream`, no allocation, no host synchronisation; nothing in the kernel waits for
 * another thread block.  Results are bit-identical from run to run.  Errors as the other calls
 * (QL_ERR_SHAPE for positions outside the cache, QL_ERR_UNSUPPORTED for other head sizes).
 * ql_attn_plan reports what a call would do: out = {first visible key, one past the last, key
 * pieces per head, 64-key sub-blocks per piece}; it needs no device.
 */
size_t ql_attn_workspace_bytes(int Hq, int Hkv);
int qattn_swa_bf16(const uint16_t* Q, const uint16_t* K, const uint16_t* V, uint16_t* out,
                   int n_q, int T, int Hq, int Hkv, int d, int p0, int window,
                   int ld_q, int ld_kv, int ld_out, void* workspace, size_t workspace_bytes, void* stream);
int ql_attn_plan(int n_q, int T, int Hq, int Hkv, int d, int p0, int window, int out[4]);

/* The stream-K split the persistent kernels use (host copies of the device arithmetic, for tests):
 * the first min(ncta, total_chunks) CTAs share an operation's chunks, CTA i owning
 * [ql_plan_first_chunk(.., i), ql_plan_first_chunk(.., i+1)); ql_plan_chunk_owner is the inverse. */
uint32_t ql_plan_first_chunk(uint32_t total_chunks, uint32_t ncta, uint32_t cta);
uint32_t ql_plan_chunk_owner(uint32_t total_chunks, uint32_t ncta, uint32_t chunk);

/* The split a CHAINED operation of n_tiles column tiles (a gate/up pair counts its double tiles)
 * and n_groups quantisation groups gets on ncta thread blocks (host copy of what the kernel
 * resolves, for tests).  range[0..1] = the chunks [lo, hi) of thread block `cta` (chunk
 * T * n_groups + G is group G of tile T); range[2] = 1 for the aligned split (at most ncta / 2 tiles
 * and at least two chunks per thread block: every tile has thread blocks of its own, and the first
 * of them, which adds the others' partial rows and finishes the tile, can be given `owner extra` chunks
 * more than an even share of the rest), 0 for the even stream-K split; range[3] = the last thread block
 * that works on the tile of chunk hi - 1.  Returns QL_OK, QL_ERR_NULL or QL_ERR_SHAPE.
 * ql_debug_set_owner_extra(e): measurement hook, process-wide, for the calls that follow: the
 * owner's extra chunks (-1: the default of 0; below -1: even split everywhere). */
int ql_plan_chain_split(int n_tiles, int n_groups, int ncta, int cta, uint32_t range[4]);
void ql_debug_set_owner_extra(int chunks);

/* Test hooks for the bounded waits of the persistent kernel (process-wide; not for production use).
 * ql_debug_set_wait_budget_ns: budget of every wait inside qlinear_stack_w4a16 launches that
 * follow (0 restores the default of 2 s).  ql_debug_no_release(i): in the launches that follow, the
 * i-th fused operation of a launch does not publish its finished tiles, so the operation after it
 * waits until its budget runs out, the status word becomes QL_ERR_DEVICE_TIMEOUT and the kernel
 * runs to its end without hanging; -1 switches the hook off.  Nothing traps or faults. */
void ql_debug_set_wait_budget_ns(uint64_t ns);
void ql_debug_no_release(int fused_op);

/* In-kernel timeline of the persistent kernel, for builds of the library with -DQL_TIMELINE
 * (ql_debug_timeline_enabled() == 1; the regular build compiles the stamps out and returns 0).
 * ql_debug_set_timeline(buf): launches that follow write globaltimer stamps (ns) into the DEVICE
 * buffer: first [160 thread blocks][n_ops][16] SM cycle stamps of thread 0 (0 operation entered,
 * 1 first chunk unpacked, 2 predecessor known complete, 3 X operand built, 4-6 first tile segment
 * drained / exchanged / published, 7 the watcher saw the predecessor complete, 8-14 the same
 * steps of the last tile segment incl. 10 polling of the contributors' rows starts, 11 partials added, 12 stores
 * issued, 14 published, 15 the publish time in globaltimer ns), then [160][4][8] cycle sums of the
 * unpack groups, [160][4][8] of the MMA issuers, and [160][n_ops] globaltimer ns at which the
 * watcher saw the predecessor complete.  paper_2607_04244_b200/timeline.py sizes and reads it.
 * NULL switches the stamps off. */
void ql_debug_set_timeline(void* device_buffer);
int ql_debug_timeline_enabled(void);

/* Timing experiments on the persistent kernel: launches that follow leave out the phases named by
 * `mask` (1 weight copies, unpacking and MMAs; 2 loading and converting the X operand; 4 waiting for
 * the row scales; 8 the exchange of split tiles; 16 the fence before a row is published; 32 the
 * accumulator exchange through shared memory; 64 the row epilogue; 256 the watcher's acquire
 * fence).  The RESULTS ARE GARBAGE while mask != 0; the step time that remains tells what the
 * left-out phases cost on the critical path.  0 restores normal operation. */
void ql_debug_set_ablate(int mask);

/* Number of kernels the library has launched since it was loaded (all entry points, this
 * process).  For benchmarks that report their launch count. */
uint64_t ql_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* QLINEAR_W4A16_H_ */
