/* libmonarch_attn — MonarchAttention forward pass (arXiv 2505.18698) for NVIDIA B200 (sm_100a).
 *
 * The method (Sec. 3 of the paper): with N = m*b, find a Monarch matrix M = P^T B whose block
 * factors L (b x m x m) and R (m x b x b) approximately maximise the softmax variational
 * objective f(M; Q, K) (Eq. 6) by T rounds of exact alternating maximisation from L = identity
 * (Eq. 7-10, R before L), then return Y = M V through the two factors (Eq. 4).  The N x N matrix
 * is never formed.
 *
 * Common conventions for every entry point
 *   - Q, K, V, Y: row-major contiguous [batch][heads][N][d]; row r of a head is block r / b,
 *     position r % b (text below Eq. 10).  Base addresses 16-byte aligned.  Y has the input
 *     dtype and must not alias an input.  All buffers are owned by the caller.
 *   - m = N / b; N must be a multiple of b; T >= 1.
 *   - softmax scale: multiplies Q (footnote to Eq. 3), i.e. both score tensors, never c_L.
 *   - Device entry points are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream).  Errors detectable on the host return before anything is enqueued.
 *   - Return value: an ma_status code.  The library never aborts and never prints.
 */
#ifndef MONARCH_ATTN_H_
#define MONARCH_ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { MA_F32 = 0, MA_F16 = 1, MA_BF16 = 2 } ma_dtype;

typedef enum {
  MA_OK = 0,
  MA_ERR_NULL = 1,        /* a required pointer is NULL */
  MA_ERR_SHAPE = 2,       /* batch, heads, N, d, b <= 0; N % b != 0; T < 1 */
  MA_ERR_DTYPE = 3,       /* dtype not one of ma_dtype */
  MA_ERR_UNSUPPORTED = 4, /* the requested path has no kernel for this (b, m, d, dtype) */
  MA_ERR_ALIGN = 5,       /* a base address is not 16-byte aligned, or Y aliases an input */
  MA_ERR_WORKSPACE = 6,   /* workspace NULL or smaller than monarch_attn_workspace_bytes() */
  MA_ERR_CUDA = 7,        /* a CUDA runtime/driver call failed */
  MA_ERR_TIMEOUT = 8,     /* a bounded device-side wait ran out (see monarch_attn_device_status) */
  MA_ERR_TOO_LARGE = 9    /* the problem needs more scratch than monarch_attn_fwd_noalloc carries */
} ma_status;

/* Which kernels run.  AUTO picks the fastest path that supports the shape. */
typedef enum {
  MA_PATH_AUTO = 0,
  MA_PATH_GENERIC = 1, /* fp32 SIMT kernels, fp32 states; any dtype, any N = m*b that fits smem */
  MA_PATH_TENSOR = 2,  /* tcgen05/TMA kernel, 16-bit states; f16/bf16, d = 64, m = b in
                          {32, 64, 128}: one persistent launch for all 2T half-steps, softmax
                          weights handed to the second MMA through shared memory; bf16 with b = 32
                          keeps alpha_L as a hi + lo pair of bf16 arrays (one more workspace
                          array).  Needs the whole GPU: see monarch_attn_fwd_ex */
  MA_PATH_TENSOR_TMEM = 3, /* the same tiles and order with the softmax weights handed over in
                              tensor memory and deeper operand rings: f16/bf16, d = 64, m = b in
                              {64, 128}.  Needs the whole GPU as well */
  MA_PATH_TENSOR_BASIC = 4,  /* one CTA per tile, one launch per half-step (no pipelining);
                                m = b in {64, 128}; the plain statement the persistent kernels are
                                tested against */
  MA_PATH_FUSED_F32 = 5, /* fp32 arithmetic and fp32 states in shared memory, one launch for all T
                            rounds: any dtype, any N = m*b whose K, V and one position's states fit
                            shared memory (N <= ~430 at d = 64); a CTA owns a set of in-block
                            positions of one head (the recursion is independent across them), so a
                            single small head is spread over up to b CTAs.  What AUTO takes for
                            fp32 inputs of that size */
  MA_PATH_FUSED_JSPLIT = 6, /* N = 1024 as m = b = 32 (d = 64, f16/bf16, either layout, no mask, no
                              row_lse): all T rounds in one launch; a head is split over four CTAs
                              by in-block position (Eq. 7-10 never mix two positions j), each
                              keeping K and its own rows of Q and of the states in shared memory.
                              f16 arithmetic with plain f16 states: what AUTO takes for T <= 2 */
  MA_PATH_FUSED_SMALL = 7, /* the same idea for any block shape: f16/bf16, m <= 32 and b <= 64 (m need
                             not equal b), d <= 64 a multiple of 8 (or b <= 32 and d <= 128), N <= 580 for T = 1 and <= 440 for
                             T > 1 (the states of a head must fit shared memory); f16 arithmetic.
                             For T >= 3 with m, b <= 16 and d <= 80 the states and the weights that
                             form them are hi + lo pairs of f16 (what AUTO takes there) */
  MA_PATH_TILE_MMA = 8    /* warp-MMA kernels, one launch per half-step, f16 states in the workspace
                             (hi + lo pairs of f16 from T = 3 on): f16/bf16, m and b <= 128 (m need
                             not equal b), d <= 128 a multiple of 8; the 16-bit path of the shapes no
                             other tensor-core kernel takes */
} ma_path;

/* T-step MonarchAttention forward (Eq. 7-10 then Eq. 4) with scale = 1/sqrt(d).
 * Q, K, V, Y: DEVICE pointers.  Uses a per-process, per-device workspace that the library grows
 * on demand (the only allocation it ever makes; call once outside any timed or captured region
 * to pre-size it).  One call in flight per device: not safe to call concurrently from several
 * host threads on one device, nor on two streams whose work may overlap (use monarch_attn_fwd_ex
 * with a workspace per stream for that; see there). */
int monarch_attn_fwd(const void* Q, const void* K, const void* V, void* Y,
                     int batch, int heads, int N, int d, int b, int T,
                     int dtype, void* stream);

/* Bytes of scratch that monarch_attn_fwd_ex needs for this problem on `path`
 * (states alpha_L, alpha_R, y, c_L, c_R of Sec. 3 'Implementation', plus a status word).
 * Returns 0 if the arguments are invalid or the path does not support them. */
size_t monarch_attn_workspace_bytes(int batch, int heads, int N, int d, int b, int T,
                                    int dtype, int path);

/* As monarch_attn_fwd, with an explicit softmax scale, an explicit path and caller-owned scratch.
 * workspace: DEVICE pointer, 256-byte aligned, at least monarch_attn_workspace_bytes() long; its
 * contents are overwritten.  Allocates nothing.
 *
 * Concurrency.  A workspace serves one call at a time: calls that may overlap on the GPU (different
 * streams, no dependency) need a workspace each, and monarch_attn_fwd's library-owned workspace
 * serves one call in flight per device.  The persistent kernels (MA_PATH_TENSOR,
 * MA_PATH_TENSOR_TMEM; what AUTO picks for d = 64, m = b in {32, 64, 128}) deal their tiles out
 * statically over one CTA per SM and the CTAs wait for each other's results, so such a launch only
 * makes progress with every CTA resident: it needs the whole GPU.  The library chains these
 * launches per device with an event, so two of them never share the SMs whatever streams they are
 * on; a foreign kernel that holds SMs for longer than the bound of the device-side waits (about a
 * second) while one of them runs makes the waits run out: the call then ends with undefined output
 * and monarch_attn_device_status reports MA_ERR_TIMEOUT. */
int monarch_attn_fwd_ex(const void* Q, const void* K, const void* V, void* Y,
                        int batch, int heads, int N, int d, int b, int T, int dtype,
                        float softmax_scale, int path,
                        void* workspace, size_t workspace_bytes, void* stream);

/* End-to-end variant: Q, K, V, Y are HOST pointers (pinned memory gives asynchronous copies).
 * Copies Q, K, V to device staging buffers owned by the library, runs monarch_attn_fwd, copies Y
 * back; does not synchronise.  The (batch, head) units are independent (Sec. 3), so the call is
 * cut into four chunks of units (measured best of 1-8 on C2 and C5): a chunk's kernels and the copy of its result run on two
 * streams owned by the library while the next chunk's inputs come in on `stream` (fork and join by
 * events, so work queued on `stream` after the call still sees Y_host complete).  Grows the staging buffers on
 * demand. */
int monarch_attn_fwd_host(const void* Q_host, const void* K_host, const void* V_host, void* Y_host,
                          int batch, int heads, int N, int d, int b, int T,
                          int dtype, void* stream);

/* Scratch the no-allocation entry point below carries inside the library image, in bytes. */
#define MONARCH_ATTN_NOALLOC_SCRATCH_BYTES (8u << 20)

/* Forward pass that also returns the value of the objective it maximises (Sec. 3, Eq. 6:
 * f(M; Q, K) = <M, scale Q K^T> + H(M); the paper reports it per iteration count as a convergence
 * diagnostic).  After the final L update, L = softmax_k Z_L exactly and every R[k,j,:] sums to one,
 * so f at the returned matrix is the sum over rows of log sum_k exp(Z_L[j,k,l]); the final L
 * half-step has that number for each row anyway and writes it out:
 *   row_lse: DEVICE pointer, [batch][heads][N] floats (natural logarithm), row b l + j of a head;
 *   f of a head = sum of its N entries (the caller reduces; 4-byte aligned).
 * `path`: MA_PATH_AUTO, MA_PATH_TENSOR (second-generation kernel), MA_PATH_FUSED_SMALL,
 * MA_PATH_TILE_MMA or MA_PATH_GENERIC.  Y, workspace
 * and everything else as monarch_attn_fwd_ex.  Asynchronous on `stream`. */
int monarch_attn_fwd_objective(const void* Q, const void* K, const void* V, void* Y, int batch,
                               int heads, int N, int d, int b, int T, int dtype,
                               float softmax_scale, int path, float* row_lse, void* workspace,
                               size_t workspace_bytes, void* stream);

/* Forward pass on tensors laid out [batch][N][heads][d] (the layout a transformer layer has after
 * its QKV projection, before any transpose); the paper's method is per head (Sec. 3), so only the
 * addressing changes.  Q, K, V, Y: DEVICE pointers to contiguous [batch][N][heads][d] arrays of
 * `dtype`, 16-byte aligned, Y not overlapping an input.  `path`: MA_PATH_AUTO, MA_PATH_TENSOR (the
 * second-generation kernel: the head becomes a column offset in the TMA tensor maps),
 * MA_PATH_FUSED_JSPLIT (likewise), MA_PATH_FUSED_SMALL, MA_PATH_FUSED_F32, MA_PATH_TILE_MMA or
 * MA_PATH_GENERIC; other paths give MA_ERR_UNSUPPORTED.  Workspace as for monarch_attn_fwd_ex with
 * the same path (monarch_attn_workspace_bytes does not depend on the layout).  Everything else as
 * monarch_attn_fwd_ex.  Asynchronous on `stream`. */
int monarch_attn_fwd_bshd(const void* Q, const void* K, const void* V, void* Y, int batch, int N,
                          int heads, int d, int b, int T, int dtype, float softmax_scale, int path,
                          void* workspace, size_t workspace_bytes, void* stream);

/* Forward pass on a post-padded sequence (Appendix C.3 "Padding and Masking").
 *
 * When the sequence length is not a multiple of the block size, the caller pads Q, K, V with rows
 * (zeros, or any finite values) up to N = ceil(n_valid / b) * b and passes the number of real rows
 * as n_valid.  The mask of that appendix (minus infinity added to Z_R for key columns
 * b k + i >= n_valid, Eq. 7) makes every column of the Monarch matrix beyond n_valid exactly zero,
 * so padded rows of V never reach the output.  Rows n_valid .. N-1 of Y are computed from the padded
 * rows of Q and carry no meaning.
 *
 * Q, K, V, Y: DEVICE pointers, [batch][heads][N][d], same rules as monarch_attn_fwd_ex.
 * n_valid must satisfy N - b < n_valid <= N (less than one block of padding, so that every key
 * block keeps a valid key; anything else is MA_ERR_SHAPE).  n_valid == N is the unpadded pass.
 * Runs on the general fused kernel (MA_PATH_FUSED_SMALL) where that supports the shape and dtype,
 * on the second-generation tensor kernel (MA_PATH_TENSOR) for f16/bf16 with d = 64 and
 * m = b in {64, 128}, on the warp-MMA tile kernels (MA_PATH_TILE_MMA) for other 16-bit shapes they
 * support, else on the generic kernels (any dtype, m need not equal b).  Workspace: the
 * larger of monarch_attn_workspace_bytes() for MA_PATH_TENSOR and MA_PATH_GENERIC serves all three
 * (a return of 0 means that path does not apply).  Asynchronous on `stream`. */
int monarch_attn_fwd_padded(const void* Q, const void* K, const void* V, void* Y, int batch,
                            int heads, int N, int d, int b, int T, int dtype, float softmax_scale,
                            int n_valid, void* workspace, size_t workspace_bytes, void* stream);

/* Forward pass on a batch of sequences of different lengths padded to one length N (Appendix C.3
 * names the case: "batched sequences of different lengths are padded to a maximum length").
 *
 * seq_len: DEVICE pointer to `batch` ints, 4-byte aligned; entry e is the number of real rows of
 * every head of batch entry e (values outside [1, N] are clamped into it).  For each sequence:
 *   - keys b k + i >= seq_len[e] get the mask of that appendix (minus infinity on Z_R, Eq. 7);
 *   - a block lying wholly in the padding (k >= ceil(seq_len[e] / b)) has no admissible R row, and
 *     the appendix gives no formula for it.  The library's reading: such a block is absent from
 *     the sequence's problem -- no weight as a key block (Z_L = -inf in Eq. 8, so every row of the
 *     Monarch matrix still sums to one over the valid keys), no term in the sums over l of Eq. 9
 *     as a query block -- so that rows 0 .. seq_len[e]-1 of Y equal what the same sequence gives
 *     when run alone at its own padded length ceil(seq_len[e] / b) * b;
 *   - rows seq_len[e] .. ceil(seq_len[e] / b) * b - 1 of Y carry no meaning, later rows are zero;
 *     rows of Q, K, V in absent blocks are never read.
 * Q, K, V, Y: DEVICE pointers, [batch][heads][N][d], rules as monarch_attn_fwd_ex.  Runs on the
 * general fused kernel (f16/bf16, short N, up to two rounds: one launch) where that applies, else
 * on the warp-MMA tile kernels (f16/bf16, m, b, d <= 128), else on the generic kernels (any dtype,
 * any N = m b); workspace: the largest of monarch_attn_workspace_bytes() for MA_PATH_FUSED_SMALL,
 * MA_PATH_TILE_MMA and MA_PATH_GENERIC.  Asynchronous on `stream`. */
int monarch_attn_fwd_varlen(const void* Q, const void* K, const void* V, void* Y, int batch,
                            int heads, int N, int d, int b, int T, int dtype, float softmax_scale,
                            const int* seq_len, void* workspace, size_t workspace_bytes,
                            void* stream);

/* The same forward pass for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of the library, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a memory pool that owns
 * the whole device, in a real-time loop where an allocation's implicit synchronisation is not
 * acceptable, or in a process whose allocator hooks forbid foreign allocations -- and that has no
 * spare buffer to lend as the workspace of monarch_attn_fwd_ex.
 *
 * What it does: runs the fp32 SIMT path (MA_PATH_GENERIC) with its states (alpha_L, alpha_R, y,
 * c_L, c_R and the status block) in a fixed MONARCH_ATTN_NOALLOC_SCRATCH_BYTES array that is part
 * of the library image; every GPU that loads the library holds that array until the process
 * exits.  Q, K, V, Y are DEVICE pointers as for monarch_attn_fwd; scale = 1/sqrt(d).
 *
 * Limits and rules:
 *   - 256 + 3*align256(4*batch*heads*N*d) + 2*align256(4*batch*heads*N) bytes must fit in the
 *     array (about batch*heads*N*d <= 690,000 for d = 64); otherwise MA_ERR_TOO_LARGE is
 *     returned and nothing is enqueued.  Shapes the generic path cannot run give
 *     MA_ERR_UNSUPPORTED.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and keeps it; make that first call before any stream capture.
 *   - It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - All calls on a device share the one array, which keeps whatever the previous call left;
 *     the status block is cleared by each call and every other word is written before it is
 *     read.  Two calls whose kernels overlap on the GPU (different streams, no dependency) race
 *     on it: serialise them. */
int monarch_attn_fwd_noalloc(const void* Q, const void* K, const void* V, void* Y,
                             int batch, int heads, int N, int d, int b, int T,
                             int dtype, void* stream);

/* Synchronises `stream` and reads the status word a run left in `workspace` (DEVICE pointer; NULL
 * means the library's own workspace on the current device): MA_OK, or MA_ERR_TIMEOUT if a bounded
 * wait inside a kernel gave up (outputs are then undefined). */
int monarch_attn_device_status(const void* workspace, void* stream);

/* Number of kernel launches the last successful call on this host thread enqueued. */
int monarch_attn_last_launch_count(void);

/* Static, NUL-terminated description of an ma_status code. */
const char* monarch_attn_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MONARCH_ATTN_H_ */
