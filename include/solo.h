/*
 * solo.h -- C ABI of the B200 (sm_100a) fused low-bit optimizer step.
 *
 * The operation is the block-wise quantized Adam(W) step of "Pushing the Limits
 * of Low-Bit Optimizers: A Focus on EMA Dynamics" (SOLO): Sec. 3.1 Eq. 2-4
 * (dequantize, EMA, quantize), Sec. 3.2.2 Eq. 6 (logarithmic quantizer with a
 * quantile-derived base for the second moment), Sec. 3.3 / Appendix A (signed
 * dynamic-exponent codebook and a precision-specific beta1 for the first moment),
 * Sec. 3.4 (4/2-bit and 2-bit Adam(W), block size 128).
 *
 * Conventions
 *   - Every pointer named *_dev or documented "device" is a CUDA device pointer
 *     of the current device; everything else is host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     All device work is enqueued on it; no call synchronizes unless it says so.
 *   - Functions return SOLO_OK (0) or a negative solo_status_t.  Nothing throws,
 *     aborts or traps on the device.  Arguments are validated on the host before
 *     anything is launched; a rejected call has no effect.
 *   - Gradients are bf16.  Parameters are fp32 or bf16 and are updated in place.
 *   - bits is 2, 3, 4 or 8 independently for the two moments; block is 64, 128,
 *     256 or 2048 elements.
 *
 * State layout (device memory owned by the solo_state_t), n_blk blocks in total,
 * tensors laid out one after the other, every tensor starting on a new block:
 *   codes_m  n_blk * block*bits_m/8 bytes   element e of a block occupies bits
 *   codes_v  n_blk * block*bits_v/8 bytes   [e*b, e*b+b) of the block's slot read
 *                                           as a little-endian bit string; a short
 *                                           last block keeps a whole slot, padding
 *                                           codes are 0
 *   scale_m  n_blk fp32   Delta of the first moment  (max |m| of the block)
 *   scale_v  n_blk fp32   Delta of the second moment (max v of the block)
 *   alpha    n_blk fp32   base of the block's logarithmic codebook, in (0,1)
 * The zero state (all codes 0, Delta = 0, alpha = 0.5) dequantizes to exact zeros.
 */
#ifndef SOLO_H_
#define SOLO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SOLO_OK = 0,
    SOLO_EINVAL = -1,   /* bad argument value (bits, block, numel, null pointer, ...) */
    SOLO_EALIGN = -2,   /* a parameter / gradient pointer is not 16-byte aligned */
    SOLO_ENOMEM = -3,   /* device or host allocation failed */
    SOLO_ECUDA = -4,    /* a CUDA runtime call or the kernel launch failed */
    SOLO_ESTATE = -5,   /* the state does not match the call (sizes, tensor count) */
    SOLO_ELIMIT = -6    /* more tensors than solo_multi_step_static has room for */
} solo_status_t;

/* Constants of the quantizers that the paper leaves open. */
#define SOLO_TINY_EXP (-100)      /* a block scale below 2^-100 is stored as 0 */
#define SOLO_RHO_MIN_EXP (-48)    /* x_p / Delta is clamped to [2^-48, 1 - 2^-10] */
#define SOLO_RHO_MAX_EXP (-10)

typedef struct solo_state solo_state_t; /* opaque; owns its device buffers */

/* Quantizers of the unsigned (second-moment) state; Appendix A gives the codebooks. */
enum {
    SOLO_V_LOG = 0,           /* levels alpha^k with the per-block base of Sec. 3.2.2 (SOLO) */
    SOLO_V_DE = 1,            /* unsigned dynamic exponent */
    SOLO_V_LINEAR = 2,        /* {0, 1/(2^b-1), ..., 1} */
    SOLO_V_LINEAR_NOZERO = 3  /* {1/2^b, ..., 1} */
};

/* Hyper-parameters of one step; plain data, read at the call and not retained. */
typedef struct {
    float lr;
    float beta1;           /* momentum of the signed EMA: the precision-specific beta' of Eq. 7 */
    float beta2;           /* momentum of the unsigned EMA (unchanged, e.g. 0.999) */
    float eps;
    float weight_decay;
    float p_quantile;      /* p of the base alpha = (x_p/Delta)^(1/(2^b-1)); 0.1 in the paper; [0,1) */
    float fixed_alpha;     /* in (0,1): every block keeps this base (standard logarithmic quantization,
                              e.g. 1/2; Sec. 3.2.2, Prop. 3.5) and no quantile is taken; else 0 */
    int32_t adamw;         /* 1: decoupled decay (AdamW); 0: decay added to the gradient (Adam) */
    int32_t bias_correction; /* 1: divide by 1-beta^t; 0: no correction */
    int32_t round_m;       /* 0: nearest level (Eq. 1); 1: stochastic rounding (Eq. 5) */
    int32_t round_v;       /* 1: xi ~ U(-1/2,1/2) in Eq. 6; 0: xi = 0 (deterministic) */
    int32_t param_dtype;   /* 0: fp32 parameters; 1: bf16 parameters */
    int32_t belief;        /* 0: Adam(W); 1: AdaBelief (Sec. 4.2): the unsigned EMA tracks
                              (g - m^)^2 and eps is added to it at every step */
    int32_t param_round;   /* bf16 parameters: 0 round to nearest even; 1 stochastic rounding with
                              the element's Philox draw (purpose 2).  No counterpart in the paper,
                              whose 16-bit baseline is plain BF16 (Sec. 4, "Baselines") */
    int32_t v_codebook;    /* quantizer of the unsigned state: SOLO_V_LOG (Eq. 6, the paper's), or
                              one of the baselines of Sec. 4 (block-wise absmax scaling, nearest
                              level of a fixed codebook, Eq. 1): SOLO_V_DE, SOLO_V_LINEAR,
                              SOLO_V_LINEAR_NOZERO.  A state must be stepped and dequantized
                              with the selector it was written with */
    uint64_t seed;         /* Philox key of the rounding noise */
} solo_hyper_t;

/*
 * Packed tensor list for solo_multi_step.  The struct itself is host memory; the
 * three arrays it points to are DEVICE memory and stay owned by the caller:
 *   param[t], grad[t]  device pointers of tensor t, each 16-byte aligned
 *   numel[t]           its element count (must equal what the state was created with)
 * `state` must come from solo_state_create_multi with the same sizes.
 */
typedef struct {
    int32_t num_tensors;
    void* const* param;          /* device array [num_tensors] of device pointers */
    const void* const* grad;     /* device array [num_tensors] of device pointers (bf16) */
    const int64_t* numel;        /* device array [num_tensors] */
    solo_state_t* state;
} solo_tensor_list_t;

/*
 * Sec. 3.4 (block-wise state of 4/2-bit and 2-bit Adam(W)).  Allocates the zero
 * state for one tensor of `numel` > 0 elements on the current device and returns
 * it in *out.  Synchronous (cudaMalloc + cudaMemset).
 */
int solo_state_create(int64_t numel, int bits_m, int bits_v, int block, solo_state_t** out);

/*
 * Same for a list of `num_tensors` tensors; numel_host is a HOST array.  Tensor t
 * owns blocks [block_start[t], block_start[t+1]) of the state, block_start being
 * the running sum of ceil(numel[t] / block).
 */
int solo_state_create_multi(const int64_t* numel_host, int num_tensors, int bits_m, int bits_v,
                            int block, solo_state_t** out);

/* Frees the state's device and host memory (synchronous).  NULL is accepted. */
int solo_state_destroy(solo_state_t* state);

/*
 * Memory accounting of Sec. 4.2 ("Block size") / Table 2: bytes of state for one
 * tensor = codes of both moments (whole slots) + 12 bytes per block.  Host only.
 */
int solo_state_bytes(int64_t numel, int bits_m, int bits_v, int block, size_t* out);

/*
 * One fused optimizer step on a single tensor (Eq. 2-4 + Adam(W), one pass over
 * HBM): per element dequantize m and v, m^ = beta1 m~ + (1-beta1) g,
 * v^ = beta2 v~ + (1-beta2) g^2, p <- p (1 - lr wd) - (lr/bc1) m^ / (sqrt(v^)/sqrt(bc2) + eps),
 * then per block the new scales, the base from the p-quantile of v^, and the new
 * codes (Eq. 1 or 5 for m, Eq. 6 for v), packed and stored.
 *   param  device, fp32 or bf16 per hyper->param_dtype, numel elements, in/out
 *   grad   device, bf16, numel elements, read only
 *   step   1-based step count t (bias corrections, Philox counter)
 * Asynchronous on `stream`.
 */
int solo_step(void* param_dev, const void* grad_dev, solo_state_t* state,
              const solo_hyper_t* hyper, int64_t step, void* stream);

/*
 * The same step over every tensor of the list, ragged block tails included, in one kernel
 * launch -- or in two when the kernel with sixteen elements per thread is selected (see
 * solo_set_kernel_policy: large sets at blocks of 64, 128 or 256; it takes the full 2048-element tiles and a
 * second, short launch the tiles that are not full; policy 2 keeps every set to one launch).
 * Tensor t uses Philox stream t.  Asynchronous on `stream`.
 */
int solo_multi_step(const solo_tensor_list_t* list, const solo_hyper_t* hyper, int64_t step,
                    void* stream);

/*
 * Sharding (Sec. 4.2, "Generalizability": optimizer states that are flattened and partitioned
 * across workers, as under FSDP, suit element-wise optimizers such as this one).  Blocks are
 * independent, so a worker may own any block-aligned piece of a tensor and step it with a state
 * of its own; the only thing that ties a piece to its tensor is the random stream of the
 * rounding noise, which is addressed by (tensor, element index).  This call tells a state where
 * each of its tensors sits in that stream; both arrays are HOST arrays of the state's tensor count:
 *   stream_id_host[t]    the number of the Philox stream of tensor t (0 .. 2^30 - 1); the
 *                        default is t, the tensor's position in the list
 *   elem_offset_host[t]  the index, within the whole tensor, of the first element that this
 *                        state's tensor t holds; a multiple of the block size; default 0
 * Either may be NULL (its default); both NULL restore the defaults.  With these set, stepping
 * the pieces of a tensor on any number of workers gives the codes, scales and parameters of
 * stepping the whole tensor at once.  Synchronizes the device; SOLO_EINVAL for an offset that is
 * negative or not on a block boundary.
 */
int solo_state_set_origin(solo_state_t* state, const int32_t* stream_id_host, const int64_t* elem_offset_host);

/*
 * The same step for a worker whose gradients arrive in HOST memory and that wants a HOST copy
 * of the updated parameters (the paper has no counterpart: it does not discuss where the
 * tensors live).  The parameters and the state stay resident on the device.  Every pointer
 * of the descriptor is a HOST array of num_tensors entries:
 *   param_dev[t]       DEVICE pointer of tensor t's parameters, 16-byte aligned, updated in place
 *   grad_host[t]       HOST pointer of its bf16 gradients (page-locked memory for overlap)
 *   param_out_host[t]  HOST pointer that receives the updated parameters (same type as the
 *                      parameters); the array may be NULL: nothing is copied back
 *   numel[t]           element counts, equal to the state's
 *   chunk_elems        elements per pipeline chunk, rounded down to whole 2048-element tiles;
 *                      0: 16 Mi
 * The tensor list is cut into chunks of whole tiles.  For each chunk the gradients are copied to
 * one of three device staging slots, the step kernel runs on the chunk's tiles, and the chunk's
 * updated parameters are copied out; each slot has its own stream, so the upload of one chunk,
 * the kernel of another and the download of a third overlap.  All of it is ordered after the
 * work queued on `stream` at the call, and `stream` waits for the last chunk.  The call itself
 * returns once all but the last three chunks have completed (it reuses page-locked staging).
 * The first call on a state, and a call with another chunk size, synchronize the device and
 * allocate the slots (3 x chunk_elems x 2 bytes) with cudaMalloc; they are freed with the state.
 * Results are identical to solo_multi_step on the same inputs.
 */
typedef struct {
    int32_t num_tensors;
    void* const* param_dev;
    const void* const* grad_host;
    void* const* param_out_host;
    const int64_t* numel;
    int64_t chunk_elems;
    solo_state_t* state;
} solo_host_list_t;
int solo_multi_step_host(const solo_host_list_t* list, const solo_hyper_t* hyper, int64_t step,
                         void* stream);

/*
 * Eq. 2 for inspection: writes the dequantized moment of every element, tensors
 * concatenated without padding (sum of numel floats).
 *   which  0: first moment y[q] * Delta_m;  1: second moment alpha^q * Delta_v, or
 *          y[q] * Delta_v with the baseline codebook of the state's last step
 *          (hyper.v_codebook; a new state decodes as SOLO_V_LOG)
 *   out_dev  device, fp32
 * Asynchronous on `stream`.
 */
int solo_dequant(const solo_state_t* state, int which, float* out_dev, void* stream);

/*
 * Raw access to the state's device buffers (tests, checkpointing).
 *   which  0 codes_m, 1 codes_v, 2 scale_m, 3 scale_v, 4 alpha
 * The pointers stay owned by the state.
 */
int solo_state_raw(const solo_state_t* state, int which, void** dev_ptr, size_t* bytes);

/* Geometry of a state: total elements, total blocks, tensors, bits, block. */
int solo_state_info(const solo_state_t* state, int64_t* numel, int64_t* num_blocks,
                    int32_t* num_tensors, int32_t* bits_m, int32_t* bits_v, int32_t* block);

/*
 * Checkpointing: the whole state as one HOST byte string, and back.  The paper stores
 * exactly these arrays (codes, block scales, bases: Sec. 3.4 and the memory accounting
 * of Table 2) but defines no file format; this one is the library's own.  Little-endian:
 *   char    magic[8] = "SOLOST1"            int32 bits_m, bits_v, block, num_tensors,
 *   int32   v_codebook, 0                   int64 num_blocks, numel[num_tensors]
 *   (padding to a multiple of 16 bytes)
 *   codes_m | codes_v | scale_m | scale_v | alpha, each padded to a multiple of 16 bytes
 * solo_state_export_bytes gives the length.  export copies device -> host on `stream`
 * and returns after the copy has completed (it synchronizes that stream); `bytes` must be
 * at least the length.  import checks that the header describes the same widths, block
 * size and tensor sizes as `state` (SOLO_ESTATE if not; SOLO_EINVAL for a short or
 * foreign buffer), copies host -> device on `stream` and also returns after completion;
 * the state then decodes and steps with the checkpoint's v_codebook.  Work queued on
 * other streams that uses the state must be ordered by the caller.
 */
int solo_state_export_bytes(const solo_state_t* state, size_t* out);
int solo_state_export(const solo_state_t* state, void* host_dst, size_t bytes, void* stream);
int solo_state_import(solo_state_t* state, const void* host_src, size_t bytes, void* stream);

/*
 * Reads the state's device status word into *status_out (0 = no problem seen).  The word is
 * sticky: bits stay set until the state is destroyed.
 *   bit 0  a solo_multi_step descriptor's numel disagreed with the state; the affected
 *          tensors were skipped
 *   bit 1  a kernel that stages its inputs gave up waiting for an asynchronous copy of them
 *          (a bounded wait, so the kernel always ends).  The warps that gave up stored nothing
 *          for the tiles concerned: those parameters and state blocks keep their old values,
 *          i.e. the step is incomplete
 * Synchronizes the device.  (No counterpart in the paper: error reporting of this library.)
 */
int solo_state_status(solo_state_t* state, int* status_out);

/*
 * Signed dynamic-exponent codebook of Appendix A (ascending, 2^bits levels) as the
 * library uses it, copied to a HOST array of 2^bits floats.
 */
int solo_codebook_m(int bits, float* levels_host);

/*
 * The same for a baseline codebook of the unsigned state (Appendix A): v_codebook is SOLO_V_DE,
 * SOLO_V_LINEAR or SOLO_V_LINEAR_NOZERO (the logarithmic levels alpha^k depend on the block and
 * have no fixed table).
 */
int solo_codebook_v(int v_codebook, int bits, float* levels_host);

/*
 * Eq. 7 with the defaults of Sec. 3.4: the recommended beta1 for `bits_m`-bit first
 * moments, from_scratch = 0 (fine-tuning, b = 5 column of Fig. 4) or 1 (b = 8 column),
 * floored to one decimal like the paper's own defaults (4 bit: 0.8 / 0.3; 2 bit: 0.5 / 0.1).
 */
float solo_default_beta1(int bits_m, int from_scratch);

/*
 * Kernel selection.  0 (default): every width and block size with the logarithmic
 * second-moment quantizer, nearest rounding of the first moment and eps >= 1e-12 runs the
 * streamlined kernel (fp32 or bf16 parameters), everything else the general one; tensor sets of
 * at least 8192 tiles of 2048 elements with 2/3/4-bit states and blocks of 64, 128 or 256 run
 * their full tiles in a kernel with sixteen elements per thread and the remaining tiles in the
 * streamlined kernel, or in the general one where the streamlined kernel does not apply (two
 * launches).  That kernel covers every mode of solo_hyper_t (Eq. 5 rounding and the baseline
 * second-moment codebooks included) as long as the quantile is the p = 0.1 one or none is taken
 * (fixed base, baseline codebook).  1: always the general kernel.  2: like 0 without the
 * sixteen-per-thread kernel.  3: like 0 with the sixteen-per-thread kernel whatever the tensor
 * sizes.  All produce the same packed state and the same bf16 parameters; the fp32 parameters
 * of the two faster kernels are identical to each other and differ from the IEEE sequence of
 * divisions and square roots by at most a few 1e-7 of the update term.  Process-wide.
 */
int solo_set_kernel_policy(int policy);

/*
 * Test hook for the streamlined kernel's rounding guard in Eq. 6: compares the hardware
 * base-2 logarithm approximation with the exact operation sequence for every binary32
 * whose bit pattern lies in [lo_bits, hi_bits] (positive normal numbers).  Writes to
 * HOST *max_excess_host the largest |approx - exact| - rel/2 * |exact| seen (or -1) and to
 * *abs_bound_host the absolute bound the kernel assumes; the guard is sound while the
 * former stays below half of the latter.  Synchronous; allocates 4 bytes of device memory.
 */
int solo_debug_check_fast_log(uint32_t lo_bits, uint32_t hi_bits, float* max_excess_host,
                              float* abs_bound_host);

/*
 * Optimizer state in buffers that the CALLER allocated (device memory), for
 * solo_multi_step_static.  Same layout as the library's own state (see the top of this
 * file): with n_blk = sum over tensors of ceil(numel / block),
 *   codes_m  n_blk * block * bits_m / 8 bytes     codes_v  n_blk * block * bits_v / 8 bytes
 *            (each followed by 16 bytes that may be read, never written)
 *   scale_m, scale_v, alpha  n_blk floats each, allocated as a multiple of 16 bytes (round
 *                            n_blk up to a multiple of 4; the padding is read, never written)
 * every buffer 16-byte aligned.  A fresh state is all-zero codes and scales and alpha = 0.5.
 */
typedef struct {
    void* codes_m;
    void* codes_v;
    float* scale_m;
    float* scale_v;
    float* alpha;
    int32_t bits_m, bits_v, block;
} solo_raw_state_t;

#define SOLO_STATIC_MAX_TENSORS 1024

/*
 * solo_multi_step for callers that must not allocate device memory.  (The paper has no
 * counterpart; this is a convenience of the library.)
 *
 * Some hosts of this step cannot call cudaMalloc at the moment they need it: code running
 * under a framework's caching allocator that wants every byte accounted for, a process whose
 * whole GPU memory was handed to a pool up front, or a step issued from a place (a stream
 * callback's consumer, a tight real-time loop) where the implicit device synchronisation of
 * cudaMalloc / cudaFree is not acceptable.  solo_state_create allocates; this entry point
 * never does.  The caller brings the state buffers (solo_raw_state_t); the small tables the
 * kernel needs besides them -- the tile and block offsets of every tensor, the first-moment
 * codebook and a status word, 32 KiB, plus 8 KiB of zeros that stand for the default position
 * of the tensors in the random stream -- live in fixed arrays inside the library that every GPU
 * loading the library holds until the process exits.
 *
 *   num_tensors        1 .. SOLO_STATIC_MAX_TENSORS; more is refused with SOLO_ELIMIT
 *   param_dev, grad_dev  DEVICE arrays of num_tensors device pointers (as in solo_tensor_list_t)
 *   numel_host         HOST array of the tensors' element counts, each > 0
 *   st                 the caller's state buffers and their geometry
 * Parameters fp32 or bf16, gradients bf16, hyper-parameters and `step` as for solo_multi_step;
 * the result is the same as solo_multi_step's on a library-owned state with equal contents.
 *
 * The fixed array is shared by every call on a device and is rewritten by each call, in
 * stream order: calls whose GPU work can overlap (different streams without ordering between
 * them) race on it and must be serialised by the caller.  Its address is looked up on the
 * first call on each device.  The call copies its tables from its own stack frame, so it must
 * not be made while `stream` is capturing: that is refused with SOLO_EINVAL before anything is
 * queued.  No cudaMalloc, cudaFree or other allocating routine is called.  Asynchronous on
 * `stream` except for the copy of the offsets from host memory, which is staged before the call
 * returns.  solo_static_status reads the call's status word.
 */
int solo_multi_step_static(int32_t num_tensors, void* const* param_dev, const void* const* grad_dev,
                           const int64_t* numel_host, const solo_raw_state_t* st,
                           const solo_hyper_t* hyper, int64_t step, void* stream);

/*
 * The status word of solo_multi_step_static's last call on the current device (same bits as
 * solo_state_status; every solo_multi_step_static call clears it before its kernels run).
 * Copies the word from the fixed array to HOST *status_out on `stream` and waits for that
 * stream; allocates nothing.  Call it on the stream the step was issued on, or after that
 * stream's work has completed.  (No counterpart in the paper.)
 */
int solo_static_status(int* status_out, void* stream);

/*
 * Test hook for the bounded wait of the kernels that stage their inputs with asynchronous
 * copies.  The next step launched by this process announces 16 bytes more than it copies for
 * the inputs of tile number `tile` (tiles of 2048 elements, counted over the tensor list), so the
 * wait for that tile's inputs runs out after its fixed number of polls: the waiting warps set
 * status bit 1, store nothing for that tile and the tiles their CTA processes after it, and the
 * kernel returns.  Nothing faults and nothing spins without limit.  One-shot and process-wide;
 * tiles that are not staged (not full, or in the general kernel) ignore it.  (No counterpart
 * in the paper.)
 */
int solo_debug_stall_copy(int64_t tile);

/* Number of kernel launches issued by this library in the calling process so far. */
int64_t solo_launch_count(void);

const char* solo_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SOLO_H_ */
