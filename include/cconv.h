/*
 * cconv -- communication-optimal direct convolution for NVIDIA B200 (sm_100a).
 *
 * C ABI of the library built from paper_1802_06905_b200/csrc (libcconv.so).
 *
 * The operation is the seven-nested-loop CNN of Demmel & Dinh, "Communication-Optimal
 * Convolutional Neural Nets" (Eq. 1, Section 2):
 *
 *     for b<B, c<C, k<K, w<W, h<H, r<R, s<S:
 *         Out(k,h,w,b) += Image(r + sw*w, s + sh*h, c, b) * Filter(k,r,s,c)
 *
 * with Out starting from zero (the library overwrites Out).  It is a cross-correlation (the filter
 * is not flipped), without padding, dilation, groups or bias.
 *
 * Array layout (the paper gives subscripts only; this ABI fixes dense row-major storage with the
 * LAST subscript fastest):
 *     Image  [Wi][Hi][C][B]   bf16,  Wi = sw*(W-1)+R,  Hi = sh*(H-1)+S  (valid-window extent)
 *     Filter [K][R][S][C]     bf16
 *     Out    [K][H][W][B]     bf16 or fp32 (h before w; Image is indexed w-direction first)
 * r runs along the first Image subscript (w-direction), s along the second (h-direction).
 * Products are accumulated in fp32.  Out is either that fp32 sum (CCONV_OUT_F32) or the sum
 * rounded once to bf16, nearest even (CCONV_OUT_BF16: one word size for all three arrays, as in
 * the paper's cost model).
 *
 * Ownership: the caller owns Image, Filter and Out.  Unless a function says "host", they are
 * DEVICE pointers on the plan's device, 16-byte aligned (Out: 32-byte aligned), and Out must not
 * overlap the inputs.
 * The library never dereferences a caller pointer after a call returns.  Device calls are
 * asynchronous on the given stream, never synchronise it, and obey stream order although their
 * kernels overlap on the GPU: per stream the library remembers the address ranges of the calls that
 * may still be running, and a call whose Image or Filter overlaps the Out of one of them, or whose
 * Out overlaps any array of one of them, starts only when the stream's earlier work is complete.
 * Independent calls (other buffers) run side by side; "kernel n complete" always implies "kernels
 * before n complete".  Calls of one explicit plan belong on one stream at a time.
 *
 * Errors: every function returns CCONV_OK (0) or a negative code; nothing throws, aborts or traps.
 * All positive loop bounds are accepted, also those outside the paper's assumptions
 * (sw <= R, sh <= S, R <= sw*W, S <= sh*H); the result is still Eq. 1.
 */
#ifndef CCONV_H_
#define CCONV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CCONV_OK 0
#define CCONV_EINVAL (-1)          /* null pointer, non-positive bound, misaligned pointer      */
#define CCONV_EUNSUPPORTED (-2)    /* requested variant cannot run this shape / this device     */
#define CCONV_ECUDA (-3)           /* a CUDA call failed; see cconv_last_cuda_error()           */
#define CCONV_EDEVICE_TIMEOUT (-4) /* a bounded device-side wait expired (kernel bug guard)     */
#define CCONV_ENOMEM (-5)
#define CCONV_ETOOLARGE (-6)       /* needs more scratch than cconv_forward_noalloc's fixed array */

/* Kernel variants (cconv_plan_create's `variant`). */
#define CCONV_VARIANT_AUTO 0
#define CCONV_VARIANT_SIMT 1 /* CUDA-core kernel: any shape, any alignment                      */
#define CCONV_VARIANT_HALO 2 /* TMA halo tiles -> tcgen05.mma -> TMEM; batch blocks of 64 or 32
                                images (the last one zero padded past B), or of 16 or 8 images     */
#define CCONV_VARIANT_STEM 3 /* small C: (s,c) folded into the MMA contraction; needs the whole
                                (shifted, padded) Filter resident in shared memory               */
#define CCONV_VARIANT_DIRECT 4 /* as HALO, but the Filter is staged straight from [K][R][S][C] by TMA:
                                  one launch per call, no scratch; b_k = 128 or 256; needs B % 8 == 0
                                  and C % 8 == 0 (no padded copies)                                */
/* The tensor-core kernels need B % 8 == 0.  For other batch sizes a plan runs them on copies of
 * Image and Out padded to the next multiple of 8 (plan-owned scratch, one padding and one compaction
 * kernel per call); for B < 8 the copies also turn bands of output rows into images, so that a
 * single image fills a block of 8 with real work (see cconv_plan_info.bands).  AUTO does so unless
 * the problem is tiny (then SIMT) or the scratch would exceed 4 GiB.  cconv_forward_noalloc, which owns no such scratch, still requires B % 8 == 0. */

/* Element type of Out (cconv_plan_create's `out_dtype`). */
#define CCONV_OUT_BF16 0
#define CCONV_OUT_F32 1

typedef struct cconv_plan cconv_plan; /* opaque; created and destroyed by the library */

typedef struct {
  /* Theorem 1 at M_words: the five terms in the paper's order, their maximum and its index 1..5 */
  double term[5];
  double bound_words;
  int bound_argmax;
  double M_words;
  /* Continuous optimum of the Section-5 tiling LP at M_words: block sizes in the order
   * b_b, b_c, b_k, b_w, b_h, b_r', b_r'', b_s', b_s''; G = their product; lp_words = F*M/G. */
  double lp_tile[9];
  double lp_G;
  double lp_words;
  /* The integer tile the kernel runs (0 where a variant has no such notion). */
  int variant;
  int out_dtype;
  int bb, bc, bk, bw, bh; /* batch, channel (per pipeline stage), out-channel, w, h block sizes */
  int halo_w, halo_h;     /* Image block extent: sw*(bw-1)+R, sh*(bh-1)+S                       */
  int stages;             /* Image shared-memory ring depth                                     */
  int filter_stages;      /* Filter shared-memory ring depth                                    */
  int grid;               /* CTAs launched (persistent kernel: <= SM count)                     */
  int tiles;              /* output tiles in total                                              */
  int smem_bytes;         /* dynamic shared memory per CTA                                      */
  int tmem_cols;          /* tensor-memory columns allocated per CTA                            */
  /* Exact traffic the integer tiling implies, in words (bf16 elements):
   * fast-memory level = shared memory of one CTA; slow side = L2/HBM. */
  double tile_words_smem; /* words staged into shared memory over the whole problem + Out words */
  double compulsory_words; /* |Image| + |Filter| + |Out| with the real Image extent             */
  /* Wave-quantisation tail (HALO variant): when the main tiling would fill its last wave of CTAs
   * only partly, output rows h >= tail_h0 run as a second launch with the tile below, started
   * while the first is in its last wave.  tail_h0 == run_H (= H unless B < 8): no tail; `tiles` and `grid` above then
   * describe the only launch, otherwise the main one. */
  int tail_h0, tail_bb, tail_bc, tail_bw, tail_bh, tail_tiles, tail_grid;
  double scratch_bytes;   /* one packed Filter; the plan owns two such device buffers and
                             alternates between them from call to call                          */
  /* What the tensor-core kernels run when B % 8 != 0 (else B, H, 1): the batch rounded up to a
   * multiple of 8 and, for B < 8, the output rows cut into `bands` bands of run_H rows, each band
   * of each image taking the place of one image (run_B = 8-multiple >= B * bands).  The tile and the
   * tail above (tail_h0 included) then describe that run. */
  int run_B, run_H, bands;
  /* HALO variant: 2 or 4 when every tile is shared by the CTAs of a cluster of that size, an equal
   * share of the channels each, partial sums exchanged through distributed shared memory (grid =
   * split * tiles; the planner does so for filters of 9 or more taps with long channel loops and few
   * output pixels), else 1. */
  int split;
  /* DIRECT variant: taps of the filter per Filter stage (a stage is filter_taps x bk x bc words). */
  int filter_taps;
  /* The paper's figure of merit for a tiling (Section 5): G = product of the block sizes, here
   * bb*bc*bk*bw*bh*R*S (the kernels never cut r and s), and its ratio to the LP optimum lp_G at
   * M_words.  bc is the channel block of one pipeline stage; the Out block stays in tensor memory
   * across all channel blocks, which the two-level model behind lp_G has no notion of. */
  double tile_G, tile_G_over_lp_G;
  /* DIRECT variant, cost model in SM cycles: lifetime of one CTA (what a call that runs alone or
   * must wait for the call in front takes) and the period of a stream of independent calls, which
   * run side by side on the SMs. */
  double est_cta_cycles, est_period_cycles;
  /* The variant that runs a call which has to wait for the stream's earlier work because its arrays
   * conflict with a call that may still be running (see the stream-order paragraph above).  AUTO
   * plans that took DIRECT, whose tiling is chosen for a stream of independent calls, keep a HALO
   * plan of the same problem for such calls, since one call alone finishes sooner on many small
   * tiles (CCONV_WAIT_TWIN=0 at plan creation: no second plan); otherwise equal to `variant`. */
  int wait_variant;
} cconv_plan_info;

/* Theorem 1 (Section 4.1): the five lower-bound terms, in words, for a fast memory of M_words.
 * Pure host arithmetic.  terms_out[0..4] = BKWH, sw*sh*BCWH, CKRS, BCKWHRS/M, BCKWH*sqrt(RS*sw*sh/M).
 * Returns CCONV_EINVAL for non-positive arguments. */
int cconv_lower_bound(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                      double M_words, double terms_out[5]);

/* Theorem 2 (Appendix A), strides 1: the leaf of the decision tree that says which expression of
 * Theorem 1 a tiling can attain for these loop bounds and a fast memory of M_words.  *leaf_out is the
 * leaf's name written as an integer (1, 21, 221, 2221, 2222 for Cases 1, 2.1, 2.2.1, 2.2.2.1,
 * 2.2.2.2); *alb_words_out (may be NULL) the attainable lower bound in words, constants dropped as
 * in the theorem.  Pure host arithmetic. */
int cconv_theorem2_case(int B, int C, int K, int W, int H, int R, int S, double M_words,
                        int* leaf_out, double* alb_words_out);

/* Section 8, "Parallel Algorithm": p processors that share one memory of M_words, the output cut
 * into aB x aK x aH x aW equal blocks (one per processor, 1 <= aX <= X).  terms_out[0..4] are the
 * five terms of the resulting bound on the total traffic: Theorem 1's, with the Image term times aK
 * and the Filter term times aB*aH*aW.  Pure host arithmetic. */
int cconv_parallel_lower_bound(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                               double M_words, int aB, int aK, int aH, int aW, double terms_out[5]);

/* The cut for p processors (1 <= p <= 65536): among all (aB, aK, aH, aW) with aX <= X and product
 * <= p, the one that uses the most processors, then gives the smallest bound, then replicates the
 * least traffic (terms 2 + 3), then is lexicographically smallest (the paper only says to choose
 * the values that minimise the bound).  a_out = {aB, aK, aH, aW}; *bound_out (may be NULL) = the
 * bound in words.  Exhaustive search on the host. */
int cconv_parallel_partition(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                             double M_words, int p, int a_out[4], double* bound_out);

/* Section 5 tiling LP (maximise the sum of log_M block sizes subject to the block-fits-in-M
 * constraints), solved at the concrete parameters with a dense simplex.  Pure host.
 * tiles_out: b_b,b_c,b_k,b_w,b_h,b_r',b_r'',b_s',b_s'' (real numbers >= 1); *G_out their product;
 * *words_out = B*C*K*W*H*R*S * M / G.  pooling != 0 drops the Filter constraint (Section 6). */
int cconv_tiling_lp(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                    double M_words, int pooling, double tiles_out[9], double* G_out,
                    double* words_out);

/* Plan: evaluate the bound, solve the LP, pick a hardware-legal tile and kernel variant for
 * `device`, and build the TMA descriptors' shape data.  M_words <= 0 means "the shared memory one
 * CTA can use, in bf16 words".  variant: CCONV_VARIANT_*; out_dtype: CCONV_OUT_*.  device >= 0 is a
 * CUDA ordinal (a status word and, for the tensor-core variants, two scratch buffers for the
 * repacked Filter are allocated there; forward calls rewrite them in turn, and the repacking of
 * one call may overlap the convolution of the call before it); device = -1 plans for a nominal
 * B200 without any CUDA call, for inspection only (forward calls on such a plan return EINVAL).
 * The plan is immutable afterwards and may be used from any stream of that device, one launch at a
 * time per plan (launches of one plan share its status word). */
int cconv_plan_create(cconv_plan** plan_out, int B, int C, int K, int W, int H, int R, int S,
                      int sw, int sh, int device, double M_words, int variant, int out_dtype);
int cconv_plan_info_get(const cconv_plan* plan, cconv_plan_info* info_out);
void cconv_plan_destroy(cconv_plan* plan);

/* Eq. 1 on device buffers (layouts above), asynchronous on `cuda_stream` (a cudaStream_t, may be
 * NULL for the default stream).  The plan's device must be the current device (else CCONV_EINVAL).  Launch errors are returned; device-side guards are read back by
 * cconv_plan_status.  A forward call allocates nothing (plans allocate at creation), so it may be
 * made while the stream is being captured into a CUDA graph. */
int cconv_forward_planned(const cconv_plan* plan, const void* Image, const void* Filter, void* Out,
                          void* cuda_stream);

/* Eq. 1 with its "+=" taken at its word on an Out that already holds values:
 *   Out(k,h,w,b) <- Out(k,h,w,b) + sum_{c,r,s} Image(r+sw*w, s+sh*h, c, b) * Filter(k,r,s,c).
 * cconv_plan_reserve_accumulate allocates, once per plan, what such calls need (an fp32 array of Out's
 * shape and a twin of the plan that writes it; CCONV_ECUDA when the allocation fails) so that the
 * calls themselves allocate nothing.  cconv_forward_accumulate runs the twin's kernels into that array
 * and then one kernel that adds it to Out: the sum is formed in fp32 and rounded once to Out's type
 * (bf16: round to nearest even).  Same pointers, alignment, stream and device rules as
 * cconv_forward_planned; CCONV_EINVAL when the plan has not reserved.  Calls of one plan share the
 * fp32 array: issue them on one stream, or order them yourself. */
int cconv_plan_reserve_accumulate(cconv_plan* plan);
int cconv_forward_accumulate(const cconv_plan* plan, const void* Image, const void* Filter, void* Out,
                             void* cuda_stream);

/* Convenience: plan (variant AUTO; cached per device, stream, shape and out_dtype, and kept until
 * the process ends) and launch on the current device.  A plan owns scratch that its calls rewrite
 * (HALO, STEM: the repacked Filter, padded copies), so calls of one plan belong on one stream; the
 * cache therefore keeps a plan per stream, and two streams may run the same shape at once.  The
 * first call of a (stream, shape) pair allocates: make it outside any stream capture. */
int cconv_forward(const void* Image, const void* Filter, void* Out, int B, int C, int K, int W,
                  int H, int R, int S, int sw, int sh, int out_dtype, void* cuda_stream);

/* Eq. 1 on arrays with EXPLICIT STRIDES.  Section 2 of the paper defines the three arrays by their
 * subscripts only -- Image(x, y, c, b), Filter(k, r, s, c), Out(k, h, w, b) -- and says nothing about
 * how they lie in memory; the rest of this ABI fixes dense row-major storage (last subscript fastest).
 * This entry point takes the element stride of every subscript instead (in the order written above;
 * all positive; distinct index tuples of Out must map to distinct addresses), so the column-major
 * reading (first subscript fastest), transposed arrays and windows of larger arrays are served too:
 *   - strides equal to the dense row-major layout, pointers aligned as for cconv_forward: the planned
 *     path (cconv_forward);
 *   - Image with contiguous images (stride of b = 1) and x, y, c strides that are multiples of 8
 *     elements (16 bytes), B % 8 == 0, Filter and Out dense and aligned: the tensor-core kernels on a
 *     tensor map built from the strides (plan cached like cconv_forward's; the first call allocates);
 *   - anything else: a CUDA-core kernel, one thread per output element, threads running along the
 *     subscript of Out with the smallest stride (pointers need only their element's alignment).
 * Asynchronous on `cuda_stream`; same error codes as cconv_forward. */
int cconv_forward_strided(const void* Image, const int64_t image_strides[4], const void* Filter,
                          const int64_t filter_strides[4], void* Out, const int64_t out_strides[4],
                          int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                          int out_dtype, void* cuda_stream);

/* Eq. 1 on HOST buffers (same layouts; pinned memory gives true asynchronous copies): copies Image
 * and Filter to device staging buffers owned by the plan (allocated on first use), launches, copies
 * Out back, all on `cuda_stream`, then synchronises that stream.  Returns the device status too. */
int cconv_forward_host(cconv_plan* plan, const void* hImage, const void* hFilter, void* hOut,
                       void* cuda_stream);

/* The same without the wait, for a loop of calls: cconv_forward_host_async returns once the work is
 * queued -- the copy of Image and Filter (pinned host memory, else the copies are not asynchronous)
 * on a copy stream of the plan, the kernels on `cuda_stream`, the copy of Out back on a second copy
 * stream -- with two sets of plan-owned staging arrays (allocated on first use), so that one call's
 * copies in either direction overlap the neighbouring calls' kernels and copies in the other
 * direction.  Calls of one plan must come from one host thread at a time and use one `cuda_stream`.
 * The host buffers of a call must stay untouched, and hOut is not valid, until cconv_host_wait has
 * returned: it waits for every queued call of the plan and returns the device status like
 * cconv_forward_host.  The plan's device must be current. */
int cconv_forward_host_async(cconv_plan* plan, const void* hImage, const void* hFilter, void* hOut,
                             void* cuda_stream);
int cconv_host_wait(cconv_plan* plan, void* cuda_stream);

/* Scratch held by cconv_forward_noalloc, in bytes (the repacked Filter must fit):
 * ceil(K/128) * ceil(C/16) * R*S * 4096 <= this. */
#define CCONV_NOALLOC_MAX_SCRATCH_BYTES (8u * 1024u * 1024u)

/* (The paper has no counterpart of this entry point; it exists for deployment.)
 * Eq. 1 on device buffers for callers that cannot allocate device memory at the time of the call:
 * code running inside a CUDA-graph capture, a serving callback whose memory was handed out at
 * start-up, a process whose allocator may not be entered from this thread.  It runs the same
 * tensor-core kernels as cconv_forward_planned (HALO variant, so B % 8 == 0 is required; other
 * shapes return CCONV_EUNSUPPORTED), but keeps the repacked Filter and the status word in a fixed
 * array inside the library (CCONV_NOALLOC_MAX_SCRATCH_BYTES + 256 bytes of device memory on every
 * GPU that loads the library, held until the process exits) instead of plan-owned cudaMalloc'd
 * memory.  It calls no cudaMalloc / cudaFree and no allocating library routine; the tile is
 * planned on the stack at every call.
 *   - Shapes whose repacked Filter exceeds the array return CCONV_ETOOLARGE; nothing is launched.
 *   - The first call on each device looks up the array's device address and the device limits
 *     (with that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents: the call rewrites
 *     the Filter blocks it uses, so back-to-back calls on ONE stream are safe (and ordered against
 *     the planned calls around them like any other call), but two calls whose kernels may overlap
 *     on the GPU (different streams, no dependency) race on the array and give wrong results.
 *     Host-side, calls are serialised by a mutex.
 *   - Asynchronous on `cuda_stream` when device_status_out is NULL.  With a non-NULL
 *     device_status_out the call synchronises the stream, stores the device status word there
 *     (0 = fine, else a bit mask of the bounded waits that expired), clears it, and returns
 *     CCONV_EDEVICE_TIMEOUT if it was non-zero. */
int cconv_forward_noalloc(const void* Image, const void* Filter, void* Out, int B, int C, int K,
                          int W, int H, int R, int S, int sw, int sh, int out_dtype,
                          void* cuda_stream, int* device_status_out);
/* (No counterpart in the paper either.)  The status word of the asynchronous cconv_forward_noalloc
 * calls made so far on the current device: synchronises `cuda_stream`, stores the word in
 * *detail_out (may be NULL), clears it, and returns CCONV_EDEVICE_TIMEOUT if it was non-zero.  The
 * kernels only ever OR bits into the word, so a wait that expired in any earlier call stays
 * visible until it is read.  Allocates nothing. */
int cconv_noalloc_status(void* cuda_stream, int* detail_out);

/* ---- Pooling (Section 6) ---------------------------------------------------------------------
 * The loop nest of Eq. 1 without its Filter,
 *
 *     for b<B, c<C, k<K, w<W, h<H, r<R, s<S:   Out(k,h,w,b) (+)= Image(r + sw*w, s + sh*h, c, b)
 *
 * where a (+) b is a + b/(R*S) with Out starting from 0 (CCONV_POOL_AVG) or max(a, b) with Out
 * starting from -infinity (CCONV_POOL_MAX).  The nest is taken literally: k does not occur on the
 * right-hand side, so the reduction runs over the channel c as well as over the window (r,s), and
 * all K planes of Out receive the same values:
 *     AVG:  Out(k,h,w,b) = (1/(R*S)) * sum_{c,r,s} Image(...)       MAX:  max_{c,r,s} Image(...)
 * The usual per-channel pooling layer is the case C = K = 1 with the channels folded into B.
 * Layouts, element types and alignment are those of the convolution (Image bf16 [Wi][Hi][C][B],
 * Out [K][H][W][B] bf16 or fp32, overwritten); sums are accumulated in fp32, the maximum is exact.
 * Any positive bounds are accepted (B % 8 == 0 takes the 16-byte vector path). */
#define CCONV_POOL_AVG 0
#define CCONV_POOL_MAX 1

/* The three terms, in words, whose maximum bounds the communication of pooling (Section 6):
 * BKWH, sw*sh*BCWH, BCKWHRS/M.  Pure host arithmetic; CCONV_EINVAL for non-positive arguments. */
int cconv_pool_lower_bound(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                           double M_words, double terms_out[3]);

/* Pooling on device buffers of the current device, asynchronous on `cuda_stream`; one kernel, no
 * scratch memory, no spin waits (so there is no status word to read).  Like the convolutions it
 * overlaps independent neighbours on its stream and keeps stream order by the same address-range
 * bookkeeping (CCONV_POOL_OVERLAP=0 in the environment makes it an ordinary launch).
 * op: CCONV_POOL_*;
 * out_dtype: CCONV_OUT_*.  Returns CCONV_EINVAL for null or misaligned pointers, non-positive
 * bounds or unknown op / out_dtype, CCONV_EUNSUPPORTED when H*W*B exceeds the grid limit
 * (about 5e11 elements), CCONV_ECUDA when the launch fails. */
int cconv_pool_forward(const void* Image, void* Out, int B, int C, int K, int W, int H, int R,
                       int S, int sw, int sh, int op, int out_dtype, void* cuda_stream);

/* Synchronises `cuda_stream`, reads the plan's device status word and clears it.  Returns CCONV_OK,
 * CCONV_EDEVICE_TIMEOUT (and *detail_out = bit mask of the waits that expired) or CCONV_ECUDA. */
int cconv_plan_status(const cconv_plan* plan, void* cuda_stream, int* detail_out);

/* Diagnostics.  When the environment variable CCONV_TRACE=1 is set at plan creation, the HALO
 * kernel stamps %globaltimer (ns) at fixed points of each CTA's roles into a [grid][16] table:
 * 0 entry, 1 set-up done, 2 first Image copy issued, 3 Image producer done, 4 Filter producer done,
 * 5 first MMA issued, 6 first tile's MMAs issued, 7 all MMAs issued, 8 first accumulator ready,
 * 9 first tile stored, 10 all tiles stored, 11 exit (the DIRECT kernel stamps the same points, and
 * puts the SM's id in slot 12 and the cycles of its first tile's main loop in slot 15).  Synchronous copy to host_out (at most
 * max_u64 values); returns the number of values copied, 0 when tracing is off, or a negative code. */
int cconv_plan_trace_read(const cconv_plan* plan, unsigned long long* host_out, int max_u64);

/* Diagnostics of the stream-order bookkeeping (host logic only: nothing is launched, no pointer is
 * dereferenced).  Registers a call on `stream_key` exactly as a forward call on that stream would
 * -- the byte ranges [lo, hi) of its Image, Filter and Out (a null lo: the call has no such array),
 * how it overlaps its neighbours (0 = an ordinary launch, 1 = inputs may be read early and Out is
 * written only after every earlier call is complete, 2 = reads and writes may overlap any number of
 * earlier calls), and the SMs' worth of CTAs it keeps resident, counted by shared/tensor memory and
 * by thread slots -- and returns the hazards found against the calls that may still be running:
 * bit 0 = its Image or Filter meets an earlier Out, bit 1 = its Out meets an earlier array (checked
 * for `overlap` 2 only); a list that is full reports both.  CCONV_EINVAL for an unknown `overlap`
 * or sm_count <= 0.  A key that no real stream uses keeps the test apart from real calls. */
int cconv_stream_order_probe(void* stream_key, const void* image_lo, const void* image_hi,
                             const void* filter_lo, const void* filter_hi, const void* out_lo,
                             const void* out_hi, int overlap, double sms_by_memory,
                             double sms_by_threads, int sm_count);

const char* cconv_strerror(int code);
const char* cconv_last_cuda_error(void); /* message of the last failed CUDA call on this thread */
int cconv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CCONV_H_ */
