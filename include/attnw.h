/*
 * attnw - attention weights P = Softmax(scale * Q K^T) on NVIDIA B200 (sm_100a).
 *
 * C ABI of libattnw.so.  The operations, each a hand-written CUDA kernel:
 *
 *   attn_fused     the whole of Attention(Q, K, V) = softmax(Q K^T / sqrt(d_k)) V of Section IV in one kernel
 *   attnw_fused*   matmul + scaling + Softmax in one kernel; scores never reach HBM
 *                  (the fused kernel of Section VII of "Attention in SRAM on Tenstorrent
 *                  Grayskull"; the product is Attention's softmax(QK^T/sqrt(d_k)) of Section IV).
 *   softmax_rows*  row-wise Softmax of precomputed scores (the dedicated kernel of
 *                  Section VI-B; definition in Section VI, max subtraction of Eq. 1).
 *
 * Conventions shared by the device entry points
 *   - Every data pointer is a DEVICE pointer owned by the caller; the library neither
 *     allocates nor frees device memory in these calls.  Tensors are row-major and contiguous.
 *   - `stream` is a cudaStream_t (NULL = the legacy default stream).  Calls enqueue work and
 *     return; they do not synchronise.
 *   - The return value is an attnw_status.  Argument errors are detected on the host and
 *     nothing is launched.  ATTNW_ERR_TIMEOUT is reported by attnw_query_status() and by the *_host calls (which
 *     synchronise anyway); the asynchronous device entry points cannot know of it when they return.
 *   - Inputs must be finite.  Non-finite inputs give unspecified values in the rows they
 *     touch and never a fault.
 *   - Runs on the current CUDA device, which must be compute capability 10.x.  There is no
 *     fallback path of any kind.
 */
#ifndef ATTNW_H_
#define ATTNW_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef enum attnw_status {
    ATTNW_OK = 0,
    ATTNW_ERR_NULL_POINTER = 1, /* a required pointer is NULL                                   */
    ATTNW_ERR_BAD_SHAPE = 2,    /* a size is < 1, overflows, or scale is negative / not finite  */
    ATTNW_ERR_MISALIGNED = 3,   /* pointer not 16-byte aligned, or row pitch not 16-byte sized  */
    ATTNW_ERR_UNSUPPORTED = 4,  /* d not in {64, 128}; device is not sm_100                     */
    ATTNW_ERR_CUDA = 5,         /* a CUDA runtime / driver call failed (launch, map encode)     */
    ATTNW_ERR_TIMEOUT = 6,      /* a bounded device-side wait gave up (see attnw_query_status)  */
    ATTNW_ERR_ALIASING = 7      /* output overlaps an input in a way the kernel cannot allow    */
} attnw_status;

/*
 * attnw_fused: P[b,h,i,j] = exp(z_ij - m_i) / sum_k exp(z_ik - m_i),
 *              z_ij = scale * sum_c Q[b,h,i,c] * K[b,h,j,c],  m_i = max_j z_ij.
 * (Section IV: Attention(Q,K,V) without the product with V; Section VII: n x d_k inputs,
 *  n x n output; Eq. 1: max-subtracted Softmax over the key index j.)
 *
 *   Q, K   device, bfloat16, [B, H, N, d]                      (read only)
 *   P      device, bfloat16 (attnw_fused) or float32 (attnw_fused_f32), [B, H, N, N]; every
 *          element is written exactly once; must not overlap Q or K
 *   B,H,N  >= 1;  N*sizeof(P element) must be a multiple of 16 (N % 8 == 0 for bfloat16,
 *          N % 4 == 0 for float32);  d in {64, 128}
 *   scale  finite, >= 0 (1/sqrt(d) in the paper); applied to the scores before the max
 * Scores are accumulated in float32 on the tensor cores; max, exponentials and sums are
 * float32; only P is rounded (to nearest even for bfloat16).
 */
int attnw_fused(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, void* stream);
int attnw_fused_f32(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, void* stream);

/*
 * attnw_fused_noalloc: attnw_fused (bfloat16 P) for callers that cannot allocate device memory.  The paper has no
 * counterpart; this is a property of the library, not of the method.
 *
 * Who needs it: code that runs where cudaMalloc is not allowed or not wanted - inside a framework whose memory pool
 * owns all device memory, in a real-time loop that must not take the allocator's lock or its implicit
 * synchronisation, or in a process that has handed the rest of the GPU's memory to someone else.  attnw_fused itself
 * allocates its exchange area with cudaMalloc the first time it runs the grid-row kernel on a device; this entry
 * point never calls cudaMalloc, cudaFree or any other allocating routine.  Its exchange area is a fixed array inside
 * the library's device image (1.25 MiB, present on every GPU that loads the library until the process exits).
 *
 * Arguments, layout and result are those of attnw_fused.  Limits, each refused with a status code and no launch:
 *   N <= 4096 (ATTNW_ERR_UNSUPPORTED beyond: one group of the grid-row kernel holds at most 4096 keys), and a device
 *   on which one group fits among at most 160 resident CTAs (the array has entries for 160; a B200 uses 144 or 148).
 * First call on a device: looks up the array's device address (cudaGetSymbolAddress) and the device's properties.
 *   Make that first call before any stream capture begins.
 * Every call on a device shares the one array, which keeps what the previous call left in it; the messages carry
 *   tags that no later call repeats, so nothing has to be cleared between calls (after about 4e9 row blocks the tags
 *   start over and the call first clears the array, in stream order).  Two calls that overlap in time on one device
 *   - different streams with nothing ordering them - race on the array: order them, or use attnw_fused for one.
 */
int attnw_fused_noalloc(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, void* stream);

/*
 * attn_fused: O[b,h,i,c] = sum_j P[b,h,i,j] * V[b,h,j,c] with P as defined for attnw_fused - Attention(Q, K, V) of
 * Section IV, the product with V that Section VIII leaves as future work - in one kernel; neither the scores nor the
 * weights reach HBM.
 *
 *   Q, K, V  device, bfloat16, [B, H, N, d]                    (read only)
 *   O        device, bfloat16, [B, H, N, d]; every element is written exactly once; must not overlap Q, K or V
 *   B,H,N    >= 1 (no divisibility condition on N);  d in {64, 128};  scale finite, >= 0
 * Scores and the products with V are accumulated in float32 on the tensor cores; max, exponentials and sums are
 * float32; the weights enter the second product rounded to bfloat16 (nearest even), O is rounded to bfloat16.
 */
int attn_fused(const void* Q, const void* K, const void* V, void* O, int B, int H, int N, int d, float scale,
               void* stream);

/*
 * attnw_project_qk: the linear transformation of the inputs into queries and keys in front of the attention weights
 * (Section IV; a step the paper leaves to the vendor's matmul and names as future work in Section VIII), for all heads in
 * one launch:   Q[b,h,n,c] = sum_m X[b,n,m] * Wq[h,c,m],   K[b,h,n,c] = sum_m X[b,n,m] * Wk[h,c,m].
 *
 *   X        device, bfloat16, [B, N, d_model]                  (read only)
 *   Wq, Wk   device, bfloat16, [H, d, d_model]: row c of head h holds column c of that head's parameter matrix, i.e.
 *            the matrices are stored transposed, contiguous along d_model               (read only)
 *   Q, K     device, bfloat16, [B, H, N, d] - the layout attnw_fused and attn_fused read; every element is written
 *            exactly once; must not overlap each other or any input
 *   B,N,H    >= 1 (no divisibility condition);  d in {64, 128};  d_model >= 8, a multiple of 8 (else
 *            ATTNW_ERR_MISALIGNED), at most 2^20
 * Products are accumulated in float32 on the tensor cores over d_model in ascending blocks of 16; the results are
 * rounded to bfloat16 (nearest even).
 */
int attnw_project_qk(const void* X, const void* Wq, const void* Wk, void* Q, void* K, int B, int N, int d_model, int H,
                     int d, void* stream);

/*
 * Which kernel attn_fused uses (process-wide; the results agree within the stated tolerance):
 *   0  default: the one-pass kernel
 *   1  two-pass kernel: row maxima and sums in a first pass over the keys, normalised weights times V in a second
 *      pass that recomputes the score tiles (two exponentials and three MMA passes per element)
 *   2  one-pass kernel: the online form of Eq. 1 - running row maximum and sum, O rescaled when the maximum has
 *      grown (one exponential and two MMA passes per element), division by the row sum at the end
 * Returns ATTNW_ERR_BAD_SHAPE for any other value.
 */
int attnw_set_attn_variant(int variant);

/*
 * Which kernel attnw_fused uses (process-wide; the results are the same within the stated tolerances):
 *   0  choose by shape (default): the grid-row kernel (see 4) when P is bfloat16 and N <= 4096; the two-pass
 *      kernel otherwise (and always for attnw_fused_f32).  On a device that cannot hold a whole group of the
 *      grid-row kernel at once the older choice applies: the SRAM-resident cluster kernel, with a large call split
 *      between it and the two-pass kernel on a per-device side stream that forks from and joins `stream` with events.
 *   1  two-pass kernel: statistics pass + normalise pass that recomputes the score tiles; any N
 *   2  SRAM-resident kernel: a cluster of ceil(N/512) <= 16 CTAs keeps a 128-row block of scores in tensor
 *      memory and exchanges local row maxima and sums across CTAs, as the fused kernel of Section VII
 *      does across Tensix cores; serves bfloat16 P and N <= 8192, any other call then returns
 *      ATTNW_ERR_UNSUPPORTED
 *   3  the same kernel with the exchange the paper leaves as future work (Section VIII): the rows are dealt out to
 *      the CTAs of the cluster, the owner of a row receives its local maxima and sums, reduces them once and
 *      sends the global values to every CTA (reduce and broadcast) instead of every CTA reducing redundantly
 *   4  grid-row kernel: the SRAM-resident design on a cooperative grid of one CTA per SM.  Consecutive ceil(N/256)
 *      CTAs form a group (the cores of one grid row in Section VII) that owns a 128-row block; every CTA keeps its
 *      128 x 256 slab of scores in half of its tensor memory, so two row blocks are in flight per CTA, and the local
 *      row maxima and sums cross the group through L2 as tagged 16-byte messages in per-device exchange areas (4.7 MB)
 *      that the library allocates on first use (cudaMalloc; never inside a stream capture).  Serves bfloat16 P and
 *      N <= 4096; any other call then returns ATTNW_ERR_UNSUPPORTED.  Launches take the exchange areas in turn, so calls on
 *      different streams of one device are safe as long as fewer than four of them are in flight at once.
 * Returns ATTNW_ERR_BAD_SHAPE for any other value.
 */
int attnw_set_fused_variant(int variant);

/*
 * softmax_rows: P[i,j] = exp(S_ij - m_i) / sum_k exp(S_ik - m_i),  m_i = max_j S_ij
 * (Softmax definition of Section VI with Eq. 1; one row is read once, kept on chip, and
 *  written once - the "caching" form of Section VI-A - unless cols exceeds the on-chip tier,
 *  where the exponentials are recomputed from a second read of the row.)
 *
 *   S      device, float32, [rows, cols]                        (read only)
 *   P      device, bfloat16 (softmax_rows) or float32 (softmax_rows_f32), [rows, cols].
 *          softmax_rows_f32 accepts P == S exactly (in place); any other overlap is refused
 *   rows   >= 1;  cols >= 1 and cols % 4 == 0;  rows * cols < 2^62
 */
int softmax_rows(const void* S, void* P, long long rows, long long cols, void* stream);
int softmax_rows_f32(const void* S, void* P, long long rows, long long cols, void* stream);

/*
 * Which form of the row Softmax softmax_rows uses (process-wide; Section VI-A compares the two on its hardware):
 *   0  by row length (default): rows of up to 262144 columns are read once and kept on chip ("caching": one
 *      exponential per element) - in registers up to 8192 columns, in the shared memory of one CTA up to 24576 and
 *      of a cluster of two CTAs up to 32768, in the registers of a cluster of 3 to 16 CTAs from 45057 to 262144;
 *      rows in between and longer rows are read twice (the second time out of L2), their exponentials recomputed
 *   1  caching only: rows of up to 393216 columns are kept in the shared memory of a thread-block cluster of up to
 *      16 CTAs that exchange local maxima and sums through distributed shared memory; a call with cols > 393216
 *      returns ATTNW_ERR_UNSUPPORTED
 *   2  recomputing for every row length, nothing kept on chip: rows of up to 32768 columns are read three times
 *      (maximum; sum of exponentials; exponentials again for the output - the second and third read come from
 *      L1 / L2), longer rows twice as under 0
 *   3  recomputing from registers: rows of up to 32768 columns are read once, the SCORES are kept in registers and
 *      every exponential is computed twice (for the sum, then for the output); longer rows: ATTNW_ERR_UNSUPPORTED
 * Returns ATTNW_ERR_BAD_SHAPE for any other value.
 */
int attnw_set_rows_variant(int variant);

/*
 * The same two operations for callers whose data lives in HOST memory (Section III describes
 * the host program's write-buffer / run / read-buffer sequence).  Pointers are HOST pointers
 * (pinned memory gives the fastest copies; pageable memory works).  The call copies the
 * inputs to the device, runs the kernel and copies P back, pipelined over groups of heads
 * (or rows), and returns after the result is complete in host memory.  Device staging
 * buffers are allocated on first use, kept per device and reused; attnw_host_release()
 * frees them.  `p_is_f32` selects the element type of P (0 = bfloat16, 1 = float32).
 * Not thread-safe with respect to other *_host calls on the same device.
 */
int attnw_fused_host(const void* Q, const void* K, void* P, int B, int H, int N, int d, float scale, int p_is_f32);
int softmax_rows_host(const void* S, void* P, long long rows, long long cols, int p_is_f32);
int attnw_host_release(void);

/*
 * Device-side failure reporting.  Every wait inside the kernels is bounded (about one second); a wait that gives
 * up records a code in a per-device status word, makes the kernel unwind and return normally, and the output of
 * that launch is then undefined.
 * The word is STICKY: while it is non-zero, every later launch of the tensor-core kernels (attnw_fused*, attn_fused,
 * attnw_project_qk) and of the shared-memory and cluster tiers of softmax_rows* (rows of 8193 to 32768 and of 45057
 * to 262144 columns) returns at once WITHOUT WRITING ITS OUTPUT - the
 * call itself still returns ATTNW_OK, since it only enqueues - so that no work piles up behind a device that has
 * stopped making progress.  The register and streaming tiers of softmax_rows* have no waits and ignore the word.
 * attnw_query_status() synchronises `stream`, stores the word in *device_status (0 = no failure; otherwise
 * 0x80000000 | an implementation code naming the wait that gave up), clears it, and returns ATTNW_OK or
 * ATTNW_ERR_TIMEOUT; after it has returned ATTNW_ERR_TIMEOUT, launches work again.  attnw_fused_host and
 * softmax_rows_host read and clear the word themselves before they return.
 */
int attnw_query_status(void* stream, unsigned int* device_status);

/*
 * Self-test of the failure path (the paper has no counterpart): launches one warp that waits, for at most
 * `limit_cycles` SM clocks (1 ... 2e9), on a barrier nobody arrives on, gives up, records site code 127 in the status
 * word and returns.  Nothing else is touched and no kernel of the library is altered; afterwards the device is in the
 * sticky state described above until attnw_query_status() is called.  ATTNW_ERR_BAD_SHAPE if the limit is out of range.
 */
int attnw_selftest_wait_timeout(long long limit_cycles, void* stream);

/* Number of kernels this library has launched in the calling process since load / last reset
 * (reset = 1 returns the count and then sets it to zero). */
long long attnw_launch_count(int reset);

/* Static string for a status code; never NULL. */
const char* attnw_strerror(int code);

/* major * 10000 + minor * 100 + patch */
int attnw_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ATTNW_H_ */
