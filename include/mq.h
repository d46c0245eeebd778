/*
 * mq.h -- C ABI of the B200-native W4A8 modality-specific static-quantized (MSQ)
 * linear path of MQuant (arXiv 2502.00425).
 *
 * Conventions shared by every call
 * --------------------------------
 *  - Every function returns an int status (MQ_OK = 0, negative = error) and never
 *    throws.  mq_status_string() names a status.
 *  - Unless a parameter says "host", every pointer is DEVICE memory owned by the
 *    caller.  The library never allocates or frees device memory; scratch comes
 *    from a caller-provided workspace sized by mq_workspace_bytes().  The one piece
 *    of device memory the library itself holds is the fixed MQ_NOALLOC_WS_BYTES
 *    array behind mq_w4a8_msq_linear_noalloc (part of its device image).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *    enqueue work on it and return without synchronising, except
 *    mq_last_device_status(), which waits for the stream.
 *  - Activations are row-major [rows, cols] with a leading dimension `ld*` counted
 *    in ELEMENTS.  bf16 activations are the usual upper-16-bits-of-float32 format.
 *    Base pointers must be 16-byte aligned and the row pitches of X and Q
 *    multiples of 16 bytes, otherwise MQ_ERR_ALIGNMENT.  A bf16 Y whose row pitch is
 *    not a multiple of 16 bytes is accepted; it is written with 2-byte instead of
 *    16-byte stores.
 *  - Weights are W[N,K] (output channel x input channel), so Y = X . W^T.
 *  - Token modality is given by a segment table (Sec. 3.1, Eq. 3: the text and
 *    visual spans of the sequence each use their own static scale): row t has the
 *    modality seg_mod[i] of the first segment i with t < seg_end[i]; rows beyond the
 *    last end are text.  After AIFS (Sec. 3.1) a sequence has two segments,
 *    [visual][text]; without AIFS the same calls take one segment per span.
 *  - Quantization follows Eq. 2 with zero-point 0: codes = clamp(round(x / s)),
 *    round-to-nearest-even, int8 range [-128,127] for activations and int4 range
 *    [-8,7] for weights; activation division is a multiplication by the float32
 *    reciprocal of the static scale.
 *  - Bad arguments are rejected on the host before anything is enqueued.  Waits
 *    inside kernels are bounded; if one ever expires the kernel records
 *    MQ_ERR_TIMEOUT in the workspace status word and returns.
 */
#ifndef MQ_H_
#define MQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MQ_VERSION 1

/* status codes */
#define MQ_OK 0
#define MQ_ERR_INVALID_ARG (-1)
#define MQ_ERR_UNSUPPORTED (-2)
#define MQ_ERR_ALIGNMENT (-3)
#define MQ_ERR_CUDA (-4)
#define MQ_ERR_TIMEOUT (-5)
#define MQ_ERR_WORKSPACE (-6)

/* modalities */
#define MQ_TEXT 0
#define MQ_VISUAL 1

/* mq_linear_desc.flags */
#define MQ_FLAG_X_IS_INT8 1u /* X is already int8 codes [T,K]; skip rotation + quantization */
#define MQ_FLAG_Y_IS_F32 2u  /* write Y as float32 instead of bfloat16 */
#define MQ_FLAG_A4 4u        /* 4-bit activation codes (W4A4): clamp to [-8,7], scales from max / 7 */
#define MQ_FLAG_W8 8u        /* 8-bit weights (W8A8): W_layout from mq_pack_w8, s_w = max / 127 */

/* Size of the library-owned scratch array behind mq_w4a8_msq_linear_noalloc (4 MiB). */
#define MQ_NOALLOC_WS_BYTES 4194304

/* Rows of the weight tile and columns of the K block of the GEMM weight layout. */
#define MQ_W_TILE_N 128
#define MQ_W_TILE_K 128

typedef struct mq_segments {
  int32_t n_seg;          /* number of segments (>= 0) */
  const int32_t* seg_end; /* device, [n_seg] exclusive cumulative row ends, non-decreasing */
  const uint8_t* seg_mod; /* device, [n_seg] MQ_TEXT / MQ_VISUAL */
} mq_segments;

typedef struct mq_linear_desc {
  int32_t T;          /* rows (tokens) of X and Y, >= 0 */
  int32_t K;          /* input channels, multiple of 32 */
  int32_t N;          /* output channels, multiple of 16 */
  int32_t rot_block;  /* online Hadamard block: 0 = off, else 32..1024 power of two dividing K */
  int32_t group_size; /* weight scale group along K: 0 = one scale per output channel, 128 = group-wise */
  uint32_t flags;     /* MQ_FLAG_* */
} mq_linear_desc;

int mq_version(void);
const char* mq_status_string(int status);

/* Bytes of scratch mq_w4a8_msq_linear needs for this problem (0 on a bad desc).
 * Holds the status word, the int8 activation codes when X arrives as bf16, and
 * split-K partial accumulators for small T.  The workspace must be 256-byte aligned. */
size_t mq_workspace_bytes(const mq_linear_desc* d);

/* Bytes of the GEMM weight layout written by mq_pack_w4 / mq_repack_w4 for W[N,K]
 * (N and K padded up to the 128 x 128 weight tile). */
size_t mq_w4_layout_bytes(int32_t N, int32_t K);

/*
 * Static-scale calibration (Sec. 3.1 "single-shot calibration"; Algorithm 1 step 6(b);
 * Eq. 2: s = max|x| / (2^(b-1) - 1) with b = 8).
 * For each modality: abs-max over all rows of that modality and all K channels of the
 * values the quantizer will see -- X after the block Hadamard rotation when rot_block
 * != 0 -- divided by 127.  A modality with no rows, or whose maximum is 0, gets 1.0f.
 *   X          bf16 [T,K], leading dimension ldx
 *   amax_state device uint32[2] owned by the caller: running abs-max bit patterns
 *              (index 0 text, 1 visual).  accumulate = 0 resets it first; accumulate = 1
 *              folds this batch into what earlier calls left, so several calibration
 *              batches give one scale.
 *   s_vis_out, s_txt_out  device float[1] each, rewritten by every call.
 */
int mq_calibrate_static_scales(const void* X, int32_t T, int32_t K, int64_t ldx,
                               const mq_segments* seg, int32_t rot_block, int32_t accumulate,
                               uint32_t* amax_state, float* s_vis_out, float* s_txt_out,
                               void* stream);

/* mq_calibrate_static_scales for b-bit activations (act_bits 8 or 4): the divisor is 2^(b-1) - 1, i.e.
 * 7 for the 4-bit activations of the W4A4 setting (Sec. 4.1).  act_bits = 8 is the call above. */
int mq_calibrate_static_scales_bits(const void* X, int32_t T, int32_t K, int64_t ldx,
                                    const mq_segments* seg, int32_t rot_block, int32_t act_bits,
                                    int32_t accumulate, uint32_t* amax_state, float* s_vis_out,
                                    float* s_txt_out, void* stream);

/*
 * Weight quantization and packing (Eq. 2 with b = 4, z = 0; Algorithm 1 outputs
 * per-channel weight scales; plain round-to-nearest stands in for GPTQ).
 *   s_w[n] = max_k |W[n,k]| / 7 (1.0f for an all-zero row);
 *   q[n,k] = clamp(round_half_even(W[n,k] / s_w[n]), -8, 7).
 *   W       float32 [N,K], leading dimension ldw
 *   packed  optional (may be NULL) canonical layout uint8 [N, K/2]:
 *           byte j of row n = (q[n,2j] & 15) | ((q[n,2j+1] & 15) << 4)
 *   s_w     float32 [N]
 *   gemm_layout optional (may be NULL) opaque layout consumed by mq_w4a8_msq_linear,
 *           mq_w4_layout_bytes(N,K) bytes, 128-byte aligned; a pure permutation of the
 *           canonical nibbles, zero-padded to whole 128 x 128 tiles.
 * group_size = 128 (group-wise W4, the g = 128 setting of the weight-only comparison, App. A.12):
 * one scale per output channel AND run of 128 input channels, s = max over the group / 7; s_w is then
 * float32 [K / 128, N] (group-major: s_w[g * N + n]) and K must be a multiple of 128.  Other non-zero
 * values MQ_ERR_UNSUPPORTED.
 */
int mq_pack_w4(const float* W, int32_t N, int32_t K, int64_t ldw, int32_t group_size,
               uint8_t* packed, float* s_w, void* gemm_layout, void* stream);

/*
 * 8-bit weights for the W8A8 setting (main results table, Sec. 4.1): Eq. 2 with b = 8,
 *   s_w[n] = max_k |W[n,k]| / 127 (1.0f for an all-zero row), q = clamp(round_half_even(W / s_w), -128, 127).
 *   q_out       optional int8 [N,K] (leading dimension ldq): the codes, for inspection
 *   gemm_layout optional, mq_w8_layout_bytes(N,K) bytes, 128-byte aligned: what mq_w4a8_msq_linear reads
 *               when MQ_FLAG_W8 is set (128 x 128 tiles of 16 KB, zero-padded)
 * At least one of q_out / gemm_layout must be given.
 */
size_t mq_w8_layout_bytes(int32_t N, int32_t K);
int mq_pack_w8(const float* W, int32_t N, int32_t K, int64_t ldw, int8_t* q_out, int64_t ldq, float* s_w,
               void* gemm_layout, void* stream);

/* Canonical [N,K/2] bytes -> GEMM weight layout (same permutation as mq_pack_w4). */
int mq_repack_w4(const uint8_t* packed, int32_t N, int32_t K, void* gemm_layout, void* stream);

/* Debug inverse: int8 codes q[N,K] (leading dimension ldq) from the canonical bytes
 * (packed != NULL) or from the GEMM layout (packed == NULL, gemm_layout != NULL). */
int mq_unpack_w4(const uint8_t* packed, const void* gemm_layout, int32_t N, int32_t K,
                 int8_t* q_out, int64_t ldq, void* stream);

/*
 * Attention-Invariant Flexible Switching, token reorder (Sec. 3.1; App. A.2:
 * AIFS(1..L) = (m..n, 1..m-1, n+1..L); App. A.4 for pads).
 * direction 0 (gather): builds perm = [indices of visual-or-pad tokens in order,
 *   then indices of text tokens in order], inv_perm, *n_first_out = size of the first
 *   block, and X_out[i,:] = X[perm[i],:].
 * direction 1 (scatter back): reads the given perm and writes X_out[perm[i],:] = X[i,:]
 *   (is_visual, is_pad, inv_perm, n_first_out are ignored and may be NULL).
 *   X, X_out   bf16 [L,D] (ldx, ldo); X == X_out is rejected.  Either both NULL
 *              (index-only call) or both non-NULL.
 *   is_visual  uint8 [L]; is_pad uint8 [L] or NULL
 *   perm, inv_perm int32 [L]; n_first_out int32 [1]
 */
int mq_aifs_reorder(const void* X, void* X_out, int32_t L, int32_t D, int64_t ldx, int64_t ldo,
                    const uint8_t* is_visual, const uint8_t* is_pad, int32_t* perm,
                    int32_t* inv_perm, int32_t* n_first_out, int32_t direction, void* stream);

/*
 * Causal-mask and position remap for the reordered sequence (Eq. 5; App. A.2: rotary
 * embeddings keep the ORIGINAL token index; App. A.4: nobody attends to pads).
 *   pos_ids_out[i] = pos_ids[perm[i]]  (pos_ids NULL = 0,1,2,...)
 *   seg_end_out[2] = {n_first, L}, seg_mod_out[2] = {MQ_VISUAL, MQ_TEXT}  (may be NULL)
 *   dense_mask_out optional uint8 [L,L], 1 = row i may attend column j:
 *       perm[j] <= perm[i] and not pad[perm[j]]  (a pad row keeps its own diagonal).
 *       Rejected with MQ_ERR_UNSUPPORTED for L > 16384.
 *   n_first    device int32[1] as written by mq_aifs_reorder (needed for seg_*_out).
 */
int mq_attn_mask_remap(const int32_t* perm, const int32_t* pos_ids, const uint8_t* is_pad,
                       const int32_t* n_first, int32_t L, int32_t* pos_ids_out,
                       int32_t* seg_end_out, uint8_t* seg_mod_out, uint8_t* dense_mask_out,
                       void* stream);

/*
 * Fused online Hadamard rotation + MSQ int8 quantizer (Fig. 4(a): the transform in
 * front of the down-projection; App. A.3: H_2, H_{2^n} = H_2 (x) H_{2^(n-1)}, applied
 * here block-diagonally over consecutive blocks of rot_block channels, normalised by
 * 1/sqrt(rot_block); Eq. 2 / Eq. 3 for the quantizer).
 *   r = X . blockdiag(H)  in float32: butterflies with strides 1,2,4,...,rot_block/2 in
 *       that order, then one multiply by float32(1/sqrt(rot_block));
 *   Q[t,k] = sat_int8(round_half_even(r[t,k] * (1.0f / s_mod(t)))).
 *   X bf16 [T,K] (ldx);  Q int8 [T,K] (ldq, multiple of 16)
 *   s_vis, s_txt  host floats, finite and > 0
 *   rotated_out   optional float32 [T,K] (leading dimension K) dump of r, NULL normally.
 */
int mq_fwht_quant_i8(const void* X, int32_t T, int32_t K, int64_t ldx, const mq_segments* seg,
                     float s_vis, float s_txt, int32_t rot_block, int8_t* Q, int64_t ldq,
                     float* rotated_out, void* stream);

/*
 * Full-width online rotation for K = m * 2^k, fused with the MSQ int8 quantizer.  App. A.3 defines H_{2^n} only;
 * for a K that is not a power of two (14336 = 28 * 512, 18944 = 148 * 128) the rotation of Fig. 4(a) is completed
 * in Kronecker form H_K = H_m (x) H_{K/m} with a Hadamard matrix of order m that the CALLER supplies:
 *   h_neg   device uint8 [m, m], h_neg[i * m + a] = 1 where H_m[i, a] = -1, 0 where it is +1
 *   r[t, a * n2 + j] = float32(1 / sqrt(K)) * sum_i H_m[i, a] * U[t, i, j],  n2 = K / m,
 *       U = the un-normalised butterflies (strides 1, 2, ..., n2 / 2) of every run of n2 channels of row t,
 *       the sum added one term at a time for i = 0, 1, ..., m - 1 in float32;
 *   Q as in mq_fwht_quant_i8;  rotated_out optional float32 [T, K] dump of r.
 * m <= 256, K / m a power of two in [32, 1024], 4 K + m^2 <= 200 KiB (the row is kept in shared memory);
 * otherwise MQ_ERR_UNSUPPORTED / MQ_ERR_INVALID_ARG.  The codes feed mq_w4a8_msq_linear with
 * MQ_FLAG_X_IS_INT8; the weight is rotated offline with the same matrix.  Cost: m additions per element.
 */
int mq_kron_quant_i8(const void* X, int32_t T, int32_t K, int64_t ldx, const mq_segments* seg, float s_vis,
                     float s_txt, int32_t m, const uint8_t* h_neg, int8_t* Q, int64_t ldq, float* rotated_out,
                     void* stream);

/* mq_fwht_quant_i8 with b-bit codes (act_bits 8 or 4; one byte per code either way): for 4 bits the
 * codes clamp to [-8, 7] (Eq. 2 with b = 4).  No rotated dump. */
int mq_fwht_quant_bits(const void* X, int32_t T, int32_t K, int64_t ldx, const mq_segments* seg,
                       float s_vis, float s_txt, int32_t rot_block, int32_t act_bits, int8_t* Q,
                       int64_t ldq, void* stream);

/*
 * The W4A8 MSQ linear (Sec. 3.1 MSQ + Fig. 4(a) + Eq. 2):
 *   Qx  = mq_fwht_quant_i8(X)            (skipped when MQ_FLAG_X_IS_INT8)
 *   acc[t,n] = sum_k Qx[t,k] * q_w[n,k]  (int32, exact)
 *   Y[t,n] = float(acc) * (s_mod(t) * s_w[n]) (+ bias[n]), rounded to bf16 (or float32).
 *   X        bf16 [T,K] or, with MQ_FLAG_X_IS_INT8, int8 [T,K]; leading dimension ldx
 *   W_layout GEMM weight layout from mq_pack_w4 / mq_repack_w4
 *   s_w      float32 [N];  bias float32 [N] or NULL
 *   Y        bf16 (or float32) [T,N], leading dimension ldy
 *   acc_out  optional int32 [T,N] (leading dimension N) dump of the accumulators
 *   ws       workspace of at least mq_workspace_bytes(d) bytes, 256-byte aligned
 * T = 0 is a successful no-op.
 * Neighbouring settings of the main results table (Sec. 4.1) and of the weight-only comparison
 * (App. A.12) run through the same call:
 *   MQ_FLAG_A4        W4A4: the quantizer clamps to [-8, 7] (pass scales calibrated with act_bits = 4);
 *   MQ_FLAG_W8        W8A8: W_layout / s_w from mq_pack_w8;
 *   group_size = 128  group-wise W4: s_w is [K / 128, N];
 *                       Y[t,n] = sum_g fl(float(acc_g[t,n]) * fl(s_mod(t) * s_w[g,n])) added in increasing g
 *                       (+ bias); acc_out, if given, is int32 [K / 128, T, N]: the accumulator of every group.
 *                       The group sums are folded into float registers after every K block, which costs
 *                       about half of the per-channel kernel's throughput (see DESIGN notes in the source).
 * MQ_FLAG_W8 and group_size = 128 exclude each other (MQ_ERR_UNSUPPORTED).
 * Which kernel runs is an internal choice that does not change the result: one to three
 * rows (single-sequence decode, the case the paper times with a W4A8 GEMV kernel,
 * Sec. 4.3) run rotation, quantizer and a CUDA-core GEMV in ONE kernel; more rows run the
 * quantizer kernel and the tensor-core GEMM (with split-K partial sums in ws for small T).
 * The kernels of consecutive calls on a stream overlap their prologues, and the GEMV issues
 * L2 prefetch hints for W_layout before the preceding kernel has finished; every real read
 * of X, W_layout and the scales is ordered after all earlier work on the stream.
 */
int mq_w4a8_msq_linear(const mq_linear_desc* d, const void* X, int64_t ldx,
                       const mq_segments* seg, float s_vis, float s_txt, const void* W_layout,
                       const float* s_w, const float* bias, void* Y, int64_t ldy,
                       int32_t* acc_out, void* ws, size_t ws_bytes, void* stream);

/*
 * mq_w4a8_msq_linear for callers that cannot supply a workspace.  (The paper has no
 * counterpart: this is an integration aid, not a step of the method.)
 *
 * The computation, the arguments and the results are those of mq_w4a8_msq_linear; only
 * the scratch differs.  Instead of a caller-owned workspace the call uses a fixed
 * MQ_NOALLOC_WS_BYTES array that is part of the library's device image.  It exists for
 * code that is handed only its inputs and outputs and may not, or cannot, allocate: a
 * plugin inside another runtime's inference loop, a decode step that must not risk the
 * device-wide lock or implicit synchronisation of an allocation, or a process whose device
 * memory is already owned in full by another pool.  The call performs no cudaMalloc, no
 * cudaFree and calls no allocating library routine.
 *
 *  - Limit: mq_workspace_bytes(d) must not exceed MQ_NOALLOC_WS_BYTES, otherwise
 *    MQ_ERR_WORKSPACE is returned and nothing is enqueued.  The workspace holds the int8
 *    codes (T * K bytes) and, where the launch splits K, one [T, N] int32 slice per split,
 *    so the limit depends on the shape: ask mq_workspace_bytes.  Decode-shaped problems
 *    fit (for example K = 4096, N = 13696 up to T = 256; K = 13696, N = 4096, which splits
 *    K four ways, up to T = 48 -- T = 64 there needs 5,071,104 bytes and is refused);
 *    prefill-sized ones need mq_w4a8_msq_linear.  The array occupies that much memory on
 *    every device the library is used on, until the process exits.
 *  - Set-up: the first call on each device looks up the array's device address (with that
 *    device current).  Make that first call outside any stream capture.
 *  - Sharing: every call on a device uses the same array, which keeps what the previous
 *    call left; the call re-initialises what has to start from zero.  Two calls that
 *    overlap on the GPU (different streams without an ordering between them) race on it:
 *    keep all calls on one stream or order them with events.
 *  - status_out: optional device int32[2] owned by the caller; receives {status, site} as
 *    mq_last_device_status would report them (MQ_OK / MQ_ERR_TIMEOUT), stream-ordered
 *    after the kernels.  Pass NULL to skip it.
 */
int mq_w4a8_msq_linear_noalloc(const mq_linear_desc* d, const void* X, int64_t ldx,
                               const mq_segments* seg, float s_vis, float s_txt,
                               const void* W_layout, const float* s_w, const float* bias, void* Y,
                               int64_t ldy, int32_t* acc_out, int32_t* status_out, void* stream);

/* ---- Rotation Magnitude Suppression (Sec. 3.2, Eq. 9) ------------------------------------
 *
 * Applies to a linear whose input is rotated online by I (x) H_n (the down-projection).  The
 * rotation concentrates a non-zero mean of each n-wide block of a weight row into the
 * block's FIRST rotated input channel (value sqrt(n) * mean, the relation stated between
 * Eq. 7 and Eq. 9).  Eq. 9 marks an (output channel, block) pair when that value exceeds the
 * block's largest original weight.  The remedy: split the first input channel of every
 * block off the rotated weight, zero it in the main matrix, run it as a separate small
 * product on the same activation codes, and add that product back.
 */

/* Row length (in codes) of the split part: K / rot_block rounded up to a multiple of 32, the
 * K granularity of the GEMM that multiplies it.  Returns 0 for an invalid (K, rot_block). */
size_t mq_rms_side_ld(int32_t K, int32_t rot_block);

/*
 * Eq. 9 on the UNROTATED weight W (device fp32 [N, K], row = output channel, leading
 * dimension ldw): flag[n, b] = sqrt(n_rot) * mean(W[n, b*n_rot .. +n_rot-1]) >
 * max(W[n, b*n_rot .. +n_rot-1]), evaluated in double precision.
 *   flags      device uint8 [N, K / rot_block], may be NULL
 *   count_out  device int32[1], number of flagged pairs, may be NULL (not both NULL)
 * rot_block: a power of two in [32, 1024] that divides K.  Offline, asynchronous on `stream`.
 */
int mq_rms_detect(const float* W, int32_t N, int32_t K, int64_t ldw, int32_t rot_block, uint8_t* flags,
                  int32_t* count_out, void* stream);

/*
 * mq_pack_w4 for a weight that gets the remedy.  W_rot is the ROTATED weight (device fp32
 * [N, K]).  Input channels k with k % rot_block == 0 form the split part:
 *   main part  all other channels; per-channel scale s_w[n] = max|.| / 7 over them; codes
 *              written to `packed` (canonical, may be NULL) and `gemm_layout` (may be NULL)
 *              exactly as mq_pack_w4 does, with code 0 at the split channels;
 *   split part q_side: device int8 [N, mq_rms_side_ld(K, rot_block)], one int4 code per byte
 *              (value in [-8, 7]), code b of row n = channel b*rot_block, padding codes 0;
 *              s_w_side[n] = max|.| / 7 over the split channels (1 if all 0);
 *              side_layout (may be NULL): the same codes in the GEMM weight layout, 128-byte
 *              aligned, mq_w4_layout_bytes(N, mq_rms_side_ld(K, rot_block)) bytes -- this is
 *              what mq_w4a8_msq_linear_rms reads; q_side is the inspectable form.
 * All outputs are caller-owned device memory.  Offline, asynchronous on `stream`.
 */
int mq_pack_w4_rms(const float* W_rot, int32_t N, int32_t K, int64_t ldw, int32_t rot_block, uint8_t* packed,
                   float* s_w, void* gemm_layout, int8_t* q_side, float* s_w_side, void* side_layout,
                   void* stream);

/* Workspace of mq_w4a8_msq_linear_rms: that of mq_w4a8_msq_linear plus the gathered split
 * activation codes [T, mq_rms_side_ld] (and, for small T, one more [T, N] int32 slice).
 * 0 for a descriptor the call would reject. */
size_t mq_rms_workspace_bytes(const mq_linear_desc* d);

/*
 * The W4A8 MSQ linear with the remedy (step 3: add the split part's product back):
 *   qx       = Q_int8(FWHT(X))                      as in mq_w4a8_msq_linear
 *   acc_main = qx . q_main^T                         (split channels are 0 in q_main)
 *   acc_side = qx[:, 0::rot_block] . q_side^T
 *   y32      = fl(acc_main * fl(s_a * s_w[n])) + fl(acc_side * fl(s_a * s_w_side[n])) (+ bias[n])
 *   Y        = bf16(y32), or y32 with MQ_FLAG_Y_IS_F32
 * d->rot_block must be non-zero and MQ_FLAG_X_IS_INT8 is not accepted (MQ_ERR_INVALID_ARG).
 * One GEMM launch computes both products: every output tile first accumulates the split
 * product (K = mq_rms_side_ld codes) into a second tensor-memory accumulator, then the main
 * product, and the epilogue combines them; there is no separate pass over Y.
 * W_layout / s_w / side_layout / s_w_side come from mq_pack_w4_rms.  acc_out and acc_side_out
 * (device int32 [T, N], either may be NULL) receive the two integer accumulators.  ws:
 * device, 256-byte aligned, at least mq_rms_workspace_bytes(d) (else MQ_ERR_WORKSPACE).
 * Everything else as mq_w4a8_msq_linear.  Asynchronous on `stream`.
 */
int mq_w4a8_msq_linear_rms(const mq_linear_desc* d, const void* X, int64_t ldx, const mq_segments* seg, float s_vis,
                           float s_txt, const void* W_layout, const float* s_w, const void* side_layout,
                           const float* s_w_side, const float* bias, void* Y, int64_t ldy, int32_t* acc_out,
                           int32_t* acc_side_out, void* ws, size_t ws_bytes, void* stream);

/* ---- Per-token dynamic A8: the comparison scheme -----------------------------------------
 *
 * The activation quantization that MSQ replaces (Sec. 1; the per-token dynamic column of the
 * latency comparison in Sec. 4.3): every token row is quantized with its own Eq. 2 scale
 * s_t = max_k |r[t,k]| / 127 taken from the rotated row at run time.  Provided so that the
 * static-versus-dynamic gap can be measured with otherwise identical kernels; not part of
 * the MSQ path, no segment table, no calibration.
 */

/*
 * Rotation (as mq_fwht_quant_i8) + per-token dynamic int8 quantizer.
 *   X bf16 [T,K] (ldx);  Q int8 [T,K] (ldq, multiple of 16);  s_rows device float32 [T] (out):
 *   s_rows[t] = max_k |r[t,k]| / 127 (1 for an all-zero row),
 *   Q[t,k] = sat_int8(round_half_even(r[t,k] * (1.0f / s_rows[t]))).
 * K <= 32768 (MQ_ERR_UNSUPPORTED beyond).  Asynchronous on `stream`.
 */
int mq_dynamic_quant_i8(const void* X, int32_t T, int32_t K, int64_t ldx, int32_t rot_block, int8_t* Q,
                        int64_t ldq, float* s_rows, void* stream);

/* Workspace of mq_w4a8_dynamic_linear: that of mq_w4a8_msq_linear plus T floats. */
size_t mq_dynamic_workspace_bytes(const mq_linear_desc* d);

/*
 * The W4A8 linear with per-token dynamic activation scales:
 *   Qx, s_rows = mq_dynamic_quant_i8(X);  acc = Qx . q_w^T;
 *   Y[t,n] = float(acc) * (s_rows[t] * s_w[n]) (+ bias[n]), rounded to bf16 (or float32).
 * MQ_FLAG_X_IS_INT8 is not accepted.  s_rows_out: optional device float32 [T] that receives
 * the scales (NULL: they stay in the workspace).  Everything else as mq_w4a8_msq_linear.
 */
int mq_w4a8_dynamic_linear(const mq_linear_desc* d, const void* X, int64_t ldx, const void* W_layout,
                           const float* s_w, const float* bias, void* Y, int64_t ldy, int32_t* acc_out,
                           float* s_rows_out, void* ws, size_t ws_bytes, void* stream);

/* ---- Glue of a decoder block (layer mode) ------------------------------------------------------
 *
 * Single-pass bf16 kernels (float32 arithmetic) for what sits between the linears of a block, so that a
 * sequence can flow through a whole layer on the library's own kernels: RMSNorm (App. A.14), the rotary
 * embedding on the ORIGINAL token positions that AIFS carries along (App. A.2), SwiGLU in front of the
 * down-projection (Fig. 4(a)) and the residual add.  Not part of the quantized path; attention under the
 * unified mask is mq_aifs_attention below.
 * All tensors bf16 row-major with leading dimensions in elements; rows 16-byte aligned (rotary: 4-byte).
 */
/* Y[t,:] = X[t,:] / sqrt(mean(X[t,:]^2) + eps) * gain;  D a multiple of 8, at most 16384. */
int mq_glue_rmsnorm(const void* X, int32_t T, int32_t D, int64_t ldx, const float* gain, float eps, void* Y,
                    int64_t ldy, void* stream);
/* Channel pairs (2i, 2i+1) of each of n_heads heads of width head_dim rotated by pos[t] * base^(-2i/head_dim);
 * X [L, n_heads * head_dim]; Y may be X (in place). */
int mq_glue_rope(const void* X, int32_t L, int32_t n_heads, int32_t head_dim, int64_t ldx, const int32_t* pos,
                 float base, void* Y, int64_t ldy, void* stream);
/* Y = G / (1 + exp(-G)) * U;  G, U, Y [T, M] (G and U may be column ranges of one wider array); M % 8 == 0. */
int mq_glue_swiglu(const void* G, int64_t ldg, const void* U, int64_t ldu, int32_t T, int32_t M, void* Y,
                   int64_t ldy, void* stream);
/* Y = A + B, one rounding to bf16;  [T, D], D % 8 == 0. */
int mq_glue_residual_add(const void* A, int64_t lda, const void* Bm, int64_t ldb, int32_t T, int32_t D, void* Y,
                         int64_t ldy, void* stream);

/* ---- Attention under the unified causal mask (Sec. 3.1, Eq. 4 - Eq. 5; App. A.4) --------------
 *
 * Grouped-query softmax attention of one sequence whose rows stand in AIFS order:
 *   O[i, h] = sum_j P[i, j] V[j, g(h)],  P[i, :] = softmax over the allowed j of  Q[i, h] . K[j, g(h)] / sqrt(D),
 * with g(h) = h / (n_q_heads / n_kv_heads).  Row i (original token perm[i]) may attend row j iff
 * perm[j] <= perm[i] and row j is not padded; a padded row also attends itself (its output is defined and
 * meant to be discarded).  With perm the AIFS permutation this is Eq. 5 for any interleaving of the
 * modalities, and the result equals causal attention (Eq. 4) in the original order, row for row.
 *
 * Q [L, n_q_heads * D], K, V [L, n_kv_heads * D], O [L, n_q_heads * D]: device bf16, row-major, leading
 * dimensions in elements, rows 16-byte aligned; Q and K already carry the rotary embedding.  perm: device
 * int32 [L] (mq_aifs_reorder's output).  pad_u: device uint8 [L] in AIFS order (1 = padded row) or NULL.
 * head_dim must be 128 and L at most 131072 (MQ_ERR_UNSUPPORTED otherwise).  float32 accumulation; the probabilities enter the
 * second product rounded to bf16.  ws: device scratch of mq_aifs_attention_workspace_bytes() bytes, 16-byte
 * aligned (it receives V transposed and the per-tile index bounds); status: device int32[2], zeroed by the
 * caller, receives MQ_ERR_TIMEOUT and the wait site if a bounded wait inside the kernel expires.
 * Enqueues two kernels on `stream`; nothing is allocated, retained or synchronised.
 */
size_t mq_aifs_attention_workspace_bytes(int32_t L, int32_t n_kv_heads, int32_t head_dim);
int mq_aifs_attention(const void* Q, int64_t ldq, const void* K, int64_t ldk, const void* V, int64_t ldv,
                      const int32_t* perm, const uint8_t* pad_u, int32_t L, int32_t n_q_heads, int32_t n_kv_heads,
                      int32_t head_dim, void* O, int64_t ldo, void* ws, size_t ws_bytes, int32_t* status, void* stream);

/* ---- Measurement and self-test aids (the paper has no counterpart) ------------------------- */

/*
 * Issue-rate microbenchmark of the int8 tensor-core instruction the GEMM is built on
 * (tcgen05.mma kind::i8, 128 x n_tok x 32 per instruction), with fixed operands and no loads: the
 * denominator "what the tensor pipe can do on this machine at the clock it holds" next to the
 * nominal and the bf16-derived figures.  `ctas` CTAs (one per SM up to the SM count) each issue
 * n_mma MMAs rotating over n_acc accumulators of n_tok columns (n_acc * n_tok <= 480); A comes
 * from tensor memory (a_from_smem = 0, as in the GEMM) or from shared memory (1).  commit_every > 0 adds a
 * tcgen05.commit to an mbarrier after every commit_every MMAs (the GEMM commits once per K block of four).
 *   cycles_out  device uint64 [ctas]: SM clock cycles from the first issue to the completion of
 *               the last MMA (0 if the bounded wait gave up)
 *   status      device int32 [2], zeroed by the caller: MQ_ERR_TIMEOUT + site if a wait gave up
 * int8 operations per clock and SM = 2 * 128 * n_tok * 32 * n_mma / cycles.
 */
int mq_ubench_mma_i8(int32_t n_tok, int32_t n_mma, int32_t n_acc, int32_t a_from_smem, int32_t commit_every,
                     int32_t ctas, uint64_t* cycles_out, int32_t* status, void* stream);

/*
 * Cost of the weight expander's inner step (packed int4 tile in shared memory -> sixteen-fold int8
 * codes in tensor memory), without barriers: one CTA of `warps` (4 or 8) warps runs n_iter rounds of
 *   mode 0: the 32-column tensor-memory store and its completion wait only,
 *   mode 1: the four 16-byte shared-memory loads, the nibble expansion and the store + wait,
 *   mode 2: as 1 but waiting for the stores once at the end.
 * cycles_out: device uint64 [warps], SM clock cycles per warp for all rounds.
 */
int mq_ubench_expand(int32_t n_iter, int32_t warps, int32_t mode, uint64_t* cycles_out, void* stream);

/*
 * Exercises the bounded wait that every kernel of the library uses on its mbarriers, on a barrier
 * that nothing arrives at: after limit_ns (1 .. 1e9) the wait gives up, writes
 * {MQ_ERR_TIMEOUT, site} to status (device int32 [2], zeroed by the caller) and raises the CTA's
 * abort flag; a second wait then returns at once.  The kernel returns normally: nothing faults.
 *   waited_ns_out  device uint64 [4]: {ns the first wait lasted, 1 if it (wrongly) succeeded,
 *                  ns the second wait lasted, 1 if it (wrongly) succeeded}
 */
int mq_selftest_bounded_wait(uint64_t limit_ns, int32_t site, int32_t* status, uint64_t* waited_ns_out,
                             void* stream);

/* Waits for `stream`, then returns the status word kernels left in the workspace
 * (MQ_OK or MQ_ERR_TIMEOUT) and, if site_out != NULL (host), where the wait gave up. */
int mq_last_device_status(void* ws, void* stream, int32_t* site_out);

/* Clears the status word (enqueued on `stream`). */
int mq_reset_device_status(void* ws, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MQ_H_ */
