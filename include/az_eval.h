/*
 * az_eval — batched evaluation of search-tree leaf positions on one NVIDIA B200 (sm_100a).
 *
 * The operation (Sec. 3.1 "At a new leaf, the network evaluates the position"; Sec. 3.3 requests
 * of many games are grouped into one GPU batch; App. D.1 network input and output contract):
 * a flat batch of independent chess positions goes in; for every position come out
 *   - prior probabilities over its legal moves (illegal actions masked before the softmax), and
 *   - a value for the player to move (win/draw/loss probabilities, or one tanh scalar).
 * Steps, all executed by this library's own CUDA kernels on the caller's stream:
 *   bitboards -> input planes -> 3x3 residual convolution tower (folded batch-norm, residual add,
 *   ReLU) -> policy head and value head -> legal-move-masked softmax.
 *
 * Conventions
 *   - Every function returns AZ_OK (0) or a negative AZ_ERR_* code; nothing throws or aborts.
 *   - "dev" pointers are device memory of the device that was current at az_load_net; "host"
 *     pointers are ordinary host memory.  The caller owns every buffer it passes and the stream.
 *     The az_net owns its weights and a workspace sized for arch.max_batch (freed by az_free_net).
 *   - Calls that take a stream are asynchronous on it.  Calls on one az_net must not overlap on
 *     the GPU (they share the workspace): use one az_net per stream.
 *   - There is no CPU fallback: without a usable CUDA device az_load_net fails with AZ_ERR_CUDA.
 *
 * Squares are numbered file + 8*rank (a1 = 0, b1 = 1, ..., h8 = 63).
 */
#ifndef AZ_EVAL_H
#define AZ_EVAL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AZ_ABI_VERSION 1
#define AZ_MAX_LEGAL 256        /* row stride of the legal-moves-only policy output (a chess position has at most 218 legal moves) */

enum {
    AZ_OK = 0,
    AZ_ERR_BAD_ARG = -1,          /* null pointer, negative size, misaligned buffer */
    AZ_ERR_BAD_ARCH = -2,         /* unsupported combination in az_arch */
    AZ_ERR_BAD_WEIGHTS = -3,      /* blob too short, wrong magic, header disagrees with az_arch, NaN/Inf */
    AZ_ERR_BATCH_TOO_LARGE = -4,  /* batch > arch.max_batch */
    AZ_ERR_CUDA = -5,             /* a CUDA runtime call failed (see az_last_cuda_error) */
    AZ_ERR_DEVICE_TIMEOUT = -6,   /* a bounded device-side wait ran out (see az_device_status) */
    AZ_ERR_NOT_CALIBRATED = -7,   /* FP8 tower used before az_calibrate */
    AZ_ERR_UNSUPPORTED = -8,      /* valid request that this build has no kernel for */
    AZ_ERR_BUSY = -9              /* az_submit_host: both in-flight slots are taken (az_wait_host first) */
};

enum { AZ_POLICY_PLANES73 = 0, AZ_POLICY_FLAT1858 = 1, AZ_POLICY_FROMTO1880 = 2 };
enum { AZ_VALUE_TANH = 0, AZ_VALUE_WDL = 1 };
/* Precision of the convolution tower (the heads are bf16 in every form but FP32):
 *   FP8_E4M3      e4m3 weights and activations, one number per operand
 *   INT8          unsigned 8-bit activations, signed 8-bit weights (the paper's deployed precision, Sec. 4.3.6)
 *   FP8_E4M3_X2   e4m3 weights and activations, every operand as a PAIR of e4m3 numbers (the rounded value and the
 *                 rounded remainder); a layer is three tensor-core products (value x value, remainder x value,
 *                 value x remainder).  Costs three times the e4m3 tower's products, i.e. 1.5 x the bf16 tower's
 *                 time, and is closer to the fp64 network than bf16.  See az_calibrate.
 *   FP8_E4M3_X2A  the same with pairs for the activations only (two products: the bf16 tower's time). */
enum { AZ_PREC_FP32 = 0, AZ_PREC_BF16 = 1, AZ_PREC_FP8_E4M3 = 2, AZ_PREC_INT8 = 3, AZ_PREC_FP8_E4M3_X2 = 4, AZ_PREC_FP8_E4M3_X2A = 5 };

/* Network shape.  in_planes 19 or 112; blocks >= 0 residual blocks of `channels` channels
 * (a multiple of 16); heads and precision as the enums above; max_batch sizes the workspace.
 * in_planes 52 selects the paper's own network (Sec. 3.2, 4.3, App. D.1): it goes with
 * policy_head AZ_POLICY_FROMTO1880 and value_head AZ_VALUE_WDL, see az_load_net. */
typedef struct {
    uint32_t abi_version;   /* AZ_ABI_VERSION */
    uint32_t in_planes;
    uint32_t blocks;
    uint32_t channels;
    uint32_t policy_head;
    uint32_t value_head;
    uint32_t precision;
    uint32_t max_batch;
} az_arch;

/* One position, 104 bytes.  pieces[] are absolute-colour bitboards in the order white P,N,B,R,Q,K
 * then black P,N,B,R,Q,K.  ep_square is the square behind a pawn that has just advanced two ranks
 * (64 if none).  halfmove is the fifty-move clock, repetitions the number of earlier occurrences
 * of this position in its game; both saturate at 255. */
typedef struct {
    uint64_t pieces[12];
    uint8_t stm;            /* 0 white to move, 1 black to move */
    uint8_t castling;       /* bit0 white O-O, bit1 white O-O-O, bit2 black O-O, bit3 black O-O-O */
    uint8_t ep_square;
    uint8_t halfmove;
    uint8_t repetitions;
    uint8_t pad[3];
} az_position;

/* Position with the seven boards before it (784 bytes); consumed by 112-plane networks.
 * hist_pieces[t-1] is the board t plies ago, n_hist (0..7) says how many are present. */
typedef struct {
    az_position cur;
    uint64_t hist_pieces[7][12];
    uint8_t hist_rep[7];
    uint8_t n_hist;
} az_position_h8;

/* Position with the last eight moves (128 bytes); consumed by the paper's 52-plane network.
 * move_from[t] / move_to[t]: absolute squares of the move t plies back (castling as the king's own
 * move), n_moves (0..8) says how many are present. */
typedef struct {
    az_position cur;
    uint8_t move_from[8];
    uint8_t move_to[8];
    uint8_t n_moves;
    uint8_t pad[7];
} az_position_m8;

typedef struct az_net az_net;

/* Size in bytes of one position record / of one position's outputs for a given arch. */
size_t az_position_bytes(const az_arch *arch);      /* 104 (19 planes), 784 (112 planes) or 128 (52 planes) */
size_t az_policy_size(const az_arch *arch);         /* 4672, 1858 or 1880 floats per position */
size_t az_mask_words(const az_arch *arch);          /* 73 or 30 uint64 words per position */
size_t az_value_size(const az_arch *arch);          /* 1 or 3 floats per position */
size_t az_plane_channels(const az_arch *arch);      /* channels of the encoded plane tensor: 32, 128 or 64 */

/*
 * load_net(weights, arch)  (Sec. 3.3 publication hands the actors a network; Sec. 4.3.6 and
 * App. D.3: batch-norm is folded into the convolutions on a deployment copy).
 * weights_host: `nbytes` of host memory holding the blob: a 64-byte header (8-byte magic
 * "AZNETv1\0", then uint32 version=1, in_planes, blocks, channels, policy_head, value_head,
 * tensor_count, zero padding) followed by raw little-endian float32 tensors in this order:
 *   input conv W[C][P][3][3], scale[C], bias[C];
 *   per block W1[C][C][3][3], scale1[C], bias1[C], W2[C][C][3][3], scale2[C], bias2[C];
 *   policy head: planes73 Wp[73][C], bp[73] | flat Wc[32][C], scale[32], bias[32], Wf[1858][2048], bf[1858];
 *   value head Wc[32][C], scale[32], bias[32], W1[128][2048], b1[128], W2[V][128], b2[V] (V = 1 or 3).
 * Convolution weights are [out][in][ky][kx]; "scale/bias" are the folded batch-norm
 * (y = scale*conv + bias).  Fully-connected inputs are flattened channel-major (c*64 + square).
 * The blob is copied; the caller may free it on return.  On success *out receives the network.
 *
 * The paper's own network (arch.in_planes == 52; Sec. 3.2, 4.3.3, 4.3.6, App. D.1): input planes as
 * az_encode52; scaled post-activation blocks, act(z) = min(max(z, 0), 6), the branch scale
 * 1/sqrt(blocks) already folded into scale2 / bias2; in blocks 1, 3, 5, ... the last C/4 output
 * channels of the first convolution are activated, averaged and maximised over the board, mapped
 * (means first, then maxima) by gw to 3C/4 values that are added to the other channels before their
 * activation, and the second convolution reads those 3C/4 channels only; policy = tokens (1x1
 * convolution with bias, no activation), queries and keys (linear maps of the token), score
 * q_origin . k_destination / sqrt(128) for the 1,792 pair actions, plus an offset (linear map of the
 * origin's token, one per piece: queen, rook, bishop, knight) for the 88 promotion actions, which
 * follow the pairs: origins on the seventh rank ascending, destinations origin+7, +8, +9 on the board,
 * then the piece; a promoting pawn move has only its promotion actions; value = 2-channel 1x1
 * convolution, folded normalisation, ReLU, 48 hidden units with ReLU, three logits, softmax.
 * Blob: 64-byte header ("AZPNET1\0", uint32 version = 1, blocks, channels, 128, 2, 48, tensor count),
 * then in.w[C][52][3][3] in.scale in.bias; per block w1[C][C][3][3] scale1 bias1, (odd blocks)
 * gw[3C/4][C/2], w2[C][C or 3C/4][3][3] scale2 bias2; t.w[128][C] t.b; q.w[128][128] q.b; k.w k.b;
 * o.w[4][128] o.b; v.cw[2][C] v.cscale v.cbias; v.w1[48][128] v.b1; v.w2[3][48] v.b2.
 * Built for the three sizes of the paper's ladder (App. D.3), channels == 128, 160 and 176, in bf16,
 * and for 128 and 160 with an int8 backbone (AZ_PREC_INT8; AZ_ERR_UNSUPPORTED otherwise).
 * Errors: BAD_ARG, BAD_ARCH, BAD_WEIGHTS, UNSUPPORTED, CUDA.
 */
int az_load_net(const az_arch *arch, const void *weights_host, size_t nbytes, az_net **out);

/*
 * az_load_net with options (az_load_net passes 0).
 * CTA pairs: the residual networks of 128 channels (bf16 and the 8-bit forms) and of 256 channels (bf16, more than
 * 148 positions) run their tower kernel as clusters of two CTAs on neighbouring SMs that share every tensor-core
 * product (tcgen05 .cta_group::2: 256 rows, 128 from each CTA; each CTA keeps HALF of every weight tile in its own
 * shared memory and bulk-copies only that half, so the operand traffic of the shared-memory pipe drops, for 128
 * channels from 8 to 6 KB per product, and the weight traffic from L2 halves).  The arithmetic and the results are
 * those of the one-CTA kernel, bit for bit.  Measured on B200 (same box): 128 channels bf16 9 to 12 % less time per
 * evaluation at every batch size from 256 to 4096 (batch 1024: 0.527 -> 0.480 ms), 256 channels 4 to 6 %, the 8-bit
 * forms 3 to 7 %, which is why it is the default for those shapes.
 *   AZ_LOAD_TOWER_CTA_PAIRS    insist on it: AZ_ERR_UNSUPPORTED for a shape that has no such form
 *   AZ_LOAD_TOWER_SINGLE_CTAS  never: the one-CTA kernel (comparisons, tests)
 * Both, or unknown bits: BAD_ARG.
 */
#define AZ_LOAD_TOWER_CTA_PAIRS 1u
#define AZ_LOAD_TOWER_SINGLE_CTAS 2u
int az_load_net_ex(const az_arch *arch, const void *weights_host, size_t nbytes, uint32_t flags, az_net **out);

/* Frees the network's device memory.  Null is allowed. */
void az_free_net(az_net *net);

/*
 * evaluate(positions, legal_masks) -> (policy, value)   (Sec. 3.1, Sec. 3.6, App. D.1).
 * positions_dev: `batch` records of az_position_bytes() each.
 * legal_masks_dev: [batch][az_mask_words()] uint64; bit (i & 63) of word (i >> 6) is set iff
 *   policy index i is a legal move (for the 73-plane head word p is plane p, bit s the origin).
 * policy_dev: [batch][az_policy_size()] float32 out: softmax over the legal entries, exactly 0
 *   elsewhere; a position whose mask is empty gets an all-zero row.
 * value_dev: [batch][az_value_size()] float32 out: tanh scalar, or (win, draw, loss) for the
 *   player to move.
 * Errors: BAD_ARG, BATCH_TOO_LARGE, NOT_CALIBRATED, CUDA.  batch == 0 is a no-op.
 */
int az_evaluate(az_net *net, const void *positions_dev, const uint64_t *legal_masks_dev,
                int batch, float *policy_dev, float *value_dev, void *cuda_stream);

/*
 * The same evaluation with the policy returned over the LEGAL moves only (Sec. 3.3: the search
 * receives priors for a leaf's legal moves): legal_policy_dev is [batch][AZ_MAX_LEGAL] float32 and
 * legal_counts_dev [batch] int32; row b holds counts[b] probabilities, the j-th one belonging to
 * the j-th set bit of position b's mask in ascending policy-index order; entries beyond counts[b]
 * are left untouched.  Values are the same numbers az_evaluate puts at those indices.  A search
 * worker fetches 1 KB per position instead of 7-19 KB.
 * Errors: as az_evaluate.
 */
int az_evaluate_legal(az_net *net, const void *positions_dev, const uint64_t *legal_masks_dev, int batch,
                      float *legal_policy_dev, int32_t *legal_counts_dev, float *value_dev, void *cuda_stream);

/* az_evaluate_legal with host buffers; see az_evaluate_host. */
int az_evaluate_legal_host(az_net *net, const void *positions_host, const uint64_t *legal_masks_host, int batch,
                           float *legal_policy_host, int32_t *legal_counts_host, float *value_host, void *cuda_stream);

/*
 * The same evaluation for callers whose buffers live in HOST memory (Sec. 5.2: preallocated
 * staging buffers, asynchronous copies and completion events between the search threads and the
 * GPU).  positions_host / legal_masks_host are copied to device staging buffers owned by the
 * az_net, the evaluation runs, policy_host / value_host receive the results, and the call returns
 * after the stream has drained.  Pinned (page-locked) host buffers make the copies asynchronous
 * with respect to other streams; pageable memory also works.  Layouts as in az_evaluate.
 * Errors: as az_evaluate.
 */
int az_evaluate_host(az_net *net, const void *positions_host, const uint64_t *legal_masks_host,
                     int batch, float *policy_host, float *value_host, void *cuda_stream);

/*
 * The encoder of the paper's own network (App. D.1, Table D.1: 52 planes).  positions_dev holds
 * 128-byte records: the 104-byte az_position, then move_from[8] and move_to[8] (absolute squares of
 * the last eight moves, most recent first, castling as the king's own move), n_moves (0..8) and
 * seven bytes of padding.  planes_dev receives [batch][64][64] float32 (bf16 == 0) or bfloat16:
 * square-major in the mover's orientation (Black to move: ranks reflected, colours exchanged,
 * files kept), channel c of the table at index c, channels 52..63 zero.
 *   0-5 own P N B R Q K, 6-11 opponent's; 12-15 castling rights own K-side, own Q-side, opponent
 *   K-side, opponent Q-side; 16, 17 all own / all opponent pieces; 18 the pieces that give check;
 *   19 the en-passant target square (set whenever the record carries one); 20, 21 one iff the
 *   position occurred at least once / twice before; 22+2t, 23+2t origin and destination of the
 *   move t plies back; 38 a checkerboard fixed in tensor coordinates with corner (0,0) set; 39 one
 *   iff each side has exactly one bishop and they stand on different colours; 40-45 own minus
 *   opponent count of P N B R Q K; 46 halfmove clock capped at 100 (a count, not normalised);
 *   47-51 own count of P N B R Q.  Every value is an integer that both output types hold exactly.
 * No az_net is involved.  Errors: BAD_ARG (null or misaligned pointer: positions 8, planes 16), CUDA.
 */
int az_encode52(const void *positions_dev, int batch, int bf16, void *planes_dev, void *cuda_stream);

/*
 * Pipelined host entry (Sec. 5.2: double-buffered staging, asynchronous copies and completion
 * events, so that the copies of one batch overlap the evaluation of the next).  az_submit_host
 * queues one evaluation and returns at once with a ticket; az_wait_host blocks until that
 * evaluation's results are in the caller's host buffers.  Up to AZ_HOST_SLOTS submissions may be
 * in flight per az_net; they run in submission order on streams the az_net owns (created on the
 * first call): the input copy of batch i+1 and the result copy of batch i-1 overlap the kernels of
 * batch i.
 *   - policy_host != NULL: dense output as az_evaluate_host (legal_policy_host / legal_counts_host
 *     ignored); policy_host == NULL: legal-moves-only output as az_evaluate_legal_host.
 *   - The host buffers must stay valid and untouched until az_wait_host returns for the ticket;
 *     pinned memory is what makes the copies asynchronous.
 *   - Tickets are small integers that are reused: wait for each ticket exactly once.
 * Errors: az_submit_host BAD_ARG, BATCH_TOO_LARGE, NOT_CALIBRATED, BUSY (nothing queued), CUDA;
 * az_wait_host BAD_ARG (no such ticket in flight), CUDA.
 */
#define AZ_HOST_SLOTS 2
int az_submit_host(az_net *net, const void *positions_host, const uint64_t *legal_masks_host, int batch,
                   float *policy_host, float *legal_policy_host, int32_t *legal_counts_host,
                   float *value_host, int *ticket);
int az_wait_host(az_net *net, int ticket);

/*
 * The encoder step alone (App. D.1: side-to-move canonical planes; for Black to move ranks are
 * reflected and colours exchanged, files keep their order).  planes_dev receives
 * [batch][64][az_plane_channels()] elements of the network's activation type (float32 for
 * AZ_PREC_FP32, bfloat16 otherwise), square-major, channels beyond in_planes zero.
 * 19 planes: 0-5 own P,N,B,R,Q,K; 6-11 opponent's; 12 one iff Black to move; 13-16 castling rights
 * own king side, own queen side, opponent king side, opponent queen side; 17 min(halfmove,100)/100;
 * 18 one iff repetitions >= 1.  112 planes: for t = 0..7 planes 13t..13t+11 the board t plies ago
 * (own then opponent, oriented by the current mover) and 13t+12 its repetition flag, zero where
 * there is no history; 104-107 castling as above; 108 one iff Black to move; 109 halfmove/100;
 * 110 zeros; 111 ones.
 */
int az_encode(az_net *net, const void *positions_dev, int batch, void *planes_dev, void *cuda_stream);

/*
 * Encoder + convolution tower alone: tower_dev receives [batch][64][channels] elements of the
 * activation type, the input of both heads (Sec. 3.5 shared backbone).  For layer-level checks.
 */
int az_tower(az_net *net, const void *positions_dev, int batch, void *tower_dev, void *cuda_stream);

/*
 * az_tower for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * entry point exists for the library's users, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits, or where a hidden allocation would
 * break a guarantee -- a plugin inside a host application that hands out all device memory from
 * its own pool and forbids others to allocate, a real-time serving thread that may not take the
 * allocator's locks or its implicit device synchronisation, or a process whose memory budget was
 * sized and frozen at start-up.  Such callers own their input and output buffers already; what they
 * lack is a way to give the library room for its intermediate plane tensor.
 *
 * This call therefore uses NO allocator at all, neither cudaMalloc / cudaFree nor any pooling
 * library: the encoded planes go to a fixed 1 MiB array that is part of the library image on the
 * device (every GPU that loads the library holds it until the process exits).  Results are the
 * same as az_tower's: tower_dev receives [batch][64][channels] bfloat16.
 *   - Limits: batch <= 256 (AZ_ERR_BATCH_TOO_LARGE beyond, and beyond arch.max_batch); networks
 *     with the bf16 tensor-core tower only, i.e. AZ_PREC_BF16, 128 channels, 19 input planes
 *     (AZ_ERR_UNSUPPORTED otherwise: fp32 networks, the 8-bit towers whether calibrated or not,
 *     other widths, the 112- and 52-plane networks).
 *   - The current device must be the one the network was loaded on (AZ_ERR_BAD_ARG otherwise):
 *     every device has its own copy of the array, and the call uses the current device's.
 *   - The first call on a device looks up the array's device address (one-time set-up under a
 *     lock, no allocation); make that first call outside any stream capture.
 *   - All calls, from every az_net and every stream, share the one array, and it keeps whatever
 *     the previous call left in it.  Nothing in it needs clearing (each call overwrites all it
 *     reads), but two calls that overlap on the GPU race on it: serialise them on one stream or
 *     with events.
 * Errors: BAD_ARG, BATCH_TOO_LARGE, UNSUPPORTED, CUDA.
 */
int az_tower_static(az_net *net, const void *positions_dev, int batch, void *tower_dev, void *cuda_stream);

/*
 * Legal-move masks from the rules of chess, computed on the GPU, in the layout az_evaluate
 * takes.  Index maps (mover-oriented coordinates; App. D.1: castling is the king-to-own-rook
 * pair, en passant the pawn's ordinary pair):
 *   planes73: index = plane*64 + origin; planes 7*d + (distance-1) for directions d =
 *     N,NE,E,SE,S,SW,W,NW; 56-63 knight jumps (1,2),(2,1),(2,-1),(1,-2),(-1,-2),(-2,-1),(-2,1),(-1,2)
 *     as (file,rank) steps; 64 + 3*piece + dir for promotion to N,B,R, dir = capture to file-1,
 *     straight, capture to file+1; queen promotion uses the one-step plane.
 *   flat1858: every (origin, destination) a queen ray or knight jump apart, origin ascending then
 *     destination ascending (1792), then for origins on the seventh rank the destinations
 *     origin+7,+8,+9 on the board, each with N,B,R (66).
 *   fromto1880 (Sec. 3.2, App. D.1): the same 1792 pairs, then the 88 promotion actions: origins on
 *     the seventh rank ascending, destinations origin+7,+8,+9 on the board, each with Q,R,B,N; a
 *     promoting pawn move sets only its four promotion actions, not the plain pair.  30 words.
 * position_stride is the byte distance between records (104, 784 or 128).  No az_net is needed.
 */
int az_legal_masks(const void *positions_dev, size_t position_stride, int batch, int policy_head,
                   uint64_t *masks_dev, void *cuda_stream);

/*
 * 8-bit towers only (AZ_PREC_FP8_E4M3, its paired forms AZ_PREC_FP8_E4M3_X2 / _X2A, AZ_PREC_INT8; Sec. 4.3.6: ranges are fixed on a few hundred
 * calibration positions): runs the bf16 tower on `n` positions, records per-channel activation
 * ranges and fixes the scales.  FP8: e4m3 activations (range / 448 per input channel, folded into
 * the weights) and e4m3 weights (one fp32 scale per output channel).  INT8, the precision the paper
 * deploys: unsigned 8-bit activations (range / 255; they are never negative), signed 8-bit weights
 * (max / 127 per output channel), int32 accumulation, the residual stream kept as int32 in the
 * second convolution's units; input layer and heads in bf16 in both.
 * Paired e4m3 forms: same scales; an activation a is stored as q1 = e4m3(a / range) and q2 = e4m3(a / range - q1)
 * (a value beyond the calibrated range saturates q1 and spills into q2), a weight likewise in _X2.
 * Then a bias correction (the usual post-training remedy for the
 * systematic part of rounding error: rounded weights meet activations that are not zero-mean, which
 * shifts every output channel's mean): layer by layer the 8-bit tower runs over the same positions
 * and the layer's biases are moved so that each channel's mean pre-activation equals the bf16
 * tower's (one tower pass per layer; shifts are limited to a quarter of the channel's range; the
 * sums behind the means are accumulated in double, so the result is repeatable).  In the paper's
 * network the pooled quarter of a pooled block's first convolution is left as it is.
 * If a CUDA error interrupts the correction, the call returns it and the network counts as not
 * calibrated again (AZ_ERR_NOT_CALIBRATED from the evaluation calls) rather than running with biases
 * corrected in part; the residual networks may then be calibrated anew, the paper's network has to
 * be loaded again (its first calibration rescales its context maps; a second one is refused with
 * AZ_ERR_UNSUPPORTED).
 * Synchronises the stream.  Errors: BAD_ARG, BATCH_TOO_LARGE, CUDA, UNSUPPORTED (not an 8-bit net).
 *
 * az_calibrate_ex is the same call with options (az_calibrate passes 0):
 *   AZ_CALIBRATE_NO_BIAS_CORRECTION  stop after the ranges and scales are fixed.  For reports that
 *     separate the rounding error of the 8-bit operands from what the correction removes.
 * Unknown bits: BAD_ARG.
 */
#define AZ_CALIBRATE_NO_BIAS_CORRECTION 1u
int az_calibrate(az_net *net, const void *positions_dev, int n, void *cuda_stream);
int az_calibrate_ex(az_net *net, const void *positions_dev, int n, uint32_t flags, void *cuda_stream);

/* Device-side status word of the last kernels (0 = clean).  Synchronises the given stream. */
int az_device_status(az_net *net, void *cuda_stream, uint32_t *status_out);

/*
 * Timing of the convolution tower alone, for roofline reports: while enabled, evaluations
 * bracket their tower kernel(s) with CUDA events on the caller's stream: every evaluation with
 * enable == 1, the k-th, 2k-th, ... after the call with enable == k > 1; 0 turns it
 * off; negative: BAD_ARG.  The events are not free: the one between the tower's launch and the head
 * kernel's keeps the latter from starting early as a dependent launch (about 9 us per evaluation at
 * batch 1024, measured), which is why a caller that also measures throughput may want k > 1.
 * az_tower_time reads the events recorded since the last read (synchronising them), returns their
 * summed duration in milliseconds and the number of bracketed tower passes, and starts afresh.  At
 * most 4096 passes are kept between reads; later ones go untimed.
 */
int az_profile_tower(az_net *net, int enable);
int az_tower_time(az_net *net, float *total_ms_out, int *passes_out);

/*
 * Self-test of the failure path: launches a one-CTA kernel whose warps wait, through the same
 * bounded wait as the tensor-core kernels, on a barrier nothing ever arrives on (poll limit a few
 * tens of microseconds).  Returns AZ_ERR_DEVICE_TIMEOUT when the wait ran out, the kernel raised its
 * status bit and still left through its normal teardown -- i.e. when failure detection works --
 * and AZ_OK / another error otherwise.  Nothing hangs or traps; the context stays usable.
 */
int az_selftest_wait_timeout(void *cuda_stream);

/* Number of kernel launches one az_evaluate of `batch` positions enqueues. */
int az_launches_per_evaluate(const az_net *net, int batch);

const char *az_strerror(int code);
/* Text of the last CUDA runtime error seen by this thread inside the library ("" if none). */
const char *az_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* AZ_EVAL_H */
