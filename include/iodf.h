/*
 * iodf.h -- C ABI of the B200 (sm_100a) integer-only discrete flow (IODF) inference library.
 *
 * The library runs the invertible integer flow of "Fast Lossless Neural Compression with
 * Integer-Only Discrete Flows" (arXiv 2206.08869) in both directions on one GPU:
 *
 *   encode  x (uint8 image batch)  ->  z (int32 latents) + prior parameters (mu, log-scale index)
 *   decode  z                      ->  x
 *
 * Every step is integer arithmetic, so both directions are exact and decode(encode(x)) == x
 * bit for bit (Sec. 3: the change of variables p_X(x) = p_Z(f(x)) needs f to be a bijection on
 * Z^d).
 *
 * Conventions
 *   - Every function returns IODF_OK (0) or a negative iodf_status; none aborts or throws.
 *   - "HOST" / "DEV" in a comment says where a pointer must live. The caller owns every buffer it
 *     passes; the library owns the model object and its device workspace.
 *   - iodf_forward / iodf_inverse enqueue work on the given CUDA stream (a cudaStream_t passed as
 *     void*; NULL = the default stream) and return without synchronising. They allocate nothing.
 *     At most one call per model may be in flight at a time (the model's workspace is shared).
 *   - All validation happens on the host before anything is launched.
 *
 * Requantisation. rq(a; M0, s) = floor((a * M0 + 2^(30+s)) / 2^(31+s)) computed exactly in 64-bit
 * integers: the fixed-point form, rounded half up, of the rescale factor s_W s_x / s_y of
 * Eq. "quant_conv" (Sec. 4.1), with M0 in [2^30, 2^31) and s in [0, 31].
 */
#ifndef IODF_H_
#define IODF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define IODF_ABI_VERSION 3u

typedef enum {
  IODF_OK = 0,
  IODF_EINVAL = -1,       /* null/misaligned pointer, batch out of range, malformed descriptor      */
  IODF_ENOMEM = -2,       /* host or device allocation failed in iodf_create                         */
  IODF_ECUDA = -3,        /* a CUDA call failed; see iodf_last_cuda_error                            */
  IODF_EVERSION = -4,     /* abi_version mismatch                                                    */
  IODF_ETIMEOUT = -5,     /* a bounded device-side wait gave up (reported by iodf_check)             */
  IODF_EUNSUPPORTED = -6, /* a valid model whose shape this build cannot run (see iodf_create)       */
  IODF_EOVERFLOW = -7,    /* a worst-case accumulator |sum| + |bias| would leave the int32 range     */
  IODF_ELIMIT = -8,       /* the request exceeds a fixed capacity (static scratch, output buffer)    */
  IODF_EDATA = -9         /* entropy coder: a scale index outside the table or a malformed stream   */
} iodf_status;

/*
 * One integer convolution layer (Eq. 5 and Eq. "quant_conv", Sec. 4.1): stride 1, zero padding
 * (k-1)/2, int8 weights and activations, int32 accumulator, int32 bias added to the accumulator,
 * then rq() per OUTPUT channel, then max(0, .) if relu, then clip to [clamp_lo, clamp_hi] if
 * has_clamp (Sec. 4.1 "Integer-Only ReLU"). Channel counts are the kept (pruned, Sec. 4.4) widths
 * and may be odd.
 */
typedef struct {
  uint32_t k;             /* kernel size: 1 or 3                                                     */
  uint32_t c_in, c_out;
  uint32_t relu;          /* 0 / 1                                                                   */
  uint32_t has_clamp;     /* 0 / 1                                                                   */
  int32_t clamp_lo, clamp_hi;
  uint64_t weight_off;    /* element offset into `weights`: int8 [c_out][k][k][c_in]                 */
  uint64_t requant_off;   /* element offset into `requant`: bias[c_out], M0[c_out], s[c_out]         */
} iodf_layer_desc;

/*
 * One residual block of a coupling network (Eq. 3, Sec. 4.1; scatter add of Sec. 4.5): how the
 * block's shortcut is requantised, how the sum is clipped, and which of the D channels of the
 * block tensor each kept output of the block's second conv is added to (see iodf_coupling_desc).
 */
typedef struct {
  int32_t short_m0, short_s;      /* shortcut requantisation Q(x) of the block, per tensor           */
  int32_t clamp_lo, clamp_hi;     /* clip after the block's ReLU                                     */
  uint32_t n_idx;                 /* = c_out of the block's second conv                              */
  const int32_t* idx;             /* HOST: channel of the D-wide block tensor that output j adds to  */
} iodf_resblock_desc;

/*
 * One additive coupling (Eq. 2, Sec. 3). Before the coupling the C channels are permuted,
 * y[k] = x[perm[k]]; x_a = y[0 : C/2] feeds the network, x_b = y[C/2 : C] is updated:
 *   a0 = clip(rq(x_a; in_m0, in_s), -128, 127);  t = layers(a0);  z_b = x_b + t  (mod 2^32).
 * The last layer must have relu = 0 and has_clamp = 0 (its rq output is the integer translation).
 *
 * With n_blocks > 0 the network is the residual form of Eq. 3 (Sec. 4.1) with the scatter add of
 * Sec. 4.5 (App. B.1: eight blocks, 3x3 convs, 128 hidden channels): layers = [conv_in,
 * (conv_a, conv_b) per block, conv_out], n_layers = 2 + 2 n_blocks. conv_in maps the requantised
 * x_a to the D-channel block tensor x (ReLU + clip); per block
 *   m = clip(ReLU(rq(conv_a(x))));  b = rq(conv_b(m))   (conv_b: relu = 0, has_clamp = 0, K' kept outputs)
 *   x = clip(max(rq(x; short_m0, short_s) [all D channels]  +  scatter of b through idx, 0), clamp_lo, clamp_hi)
 * and conv_out maps x to the integer translation. This build runs it for 3x3 convs with D and every
 * kept width <= 128, hidden activations in 0..255, and levels of at most 2048 pixels per
 * image (above 256 pixels the rows of an image are shared out over up to eight CTAs of one
 * thread-block cluster, which needs bands of at least two rows); all couplings of a level must
 * then be of this form.
 */
typedef struct {
  const int32_t* perm;            /* HOST, C entries, a permutation of 0..C-1                        */
  int32_t in_m0, in_s;
  uint32_t n_layers;
  const iodf_layer_desc* layers;  /* HOST                                                            */
  uint32_t n_blocks;              /* 0: the layers are a plain chain                                 */
  const iodf_resblock_desc* blocks; /* HOST, n_blocks entries                                        */
} iodf_coupling_desc;

/*
 * One flow level (Sec. 5 / App. B.1): a 2x2 space-to-depth (out channel c*4 + dy*2 + dx takes
 * in[c][2i+dy][2j+dx]), n_couplings couplings, then, if split, the second half of the channels is
 * factored out into z and the first half goes on. With has_prior the prior head runs on the kept
 * half: a0 = clip(rq(keep; prior_in_m0, prior_in_s), -128, 127); prior_layer maps C/2 -> 2*(C/2)
 * channels, the first half being mu (int32, unclipped) and the second the log-scale index clipped
 * to [ls_lo, ls_hi], one pair per factored-out element (Sec. 3, discretised logistic prior).
 */
typedef struct {
  uint32_t n_couplings;
  const iodf_coupling_desc* couplings; /* HOST                                                       */
  uint32_t split;
  uint32_t has_prior;                  /* requires split                                             */
  int32_t prior_in_m0, prior_in_s;
  iodf_layer_desc prior_layer;
  int32_t ls_lo, ls_hi;
} iodf_level_desc;

/* How the levels whose images are smaller than a 128-pixel tile are shared out over CTAs (the
 * results are the same bit for bit; only the launch shapes differ):
 *   IODF_PLAN_LATENCY     as few images per CTA as keeps the SMs busy with one batch of max_batch
 *                         images: the shortest step
 *   IODF_PLAN_THROUGHPUT  as many images per CTA as a tile holds with the level's weights still
 *                         resident in shared memory (levels with residual-block couplings: as many
 *                         padded frames (h+2)(w+2) as a tile holds): fewer CTAs per launch, a step a
 *                         few percent longer; for callers that keep several batches in flight, each on
 *                         a stream and a model handle of its own, so that one batch's idle SMs run
 *                         another's CTAs
 */
#define IODF_PLAN_LATENCY 0u
#define IODF_PLAN_THROUGHPUT 1u

typedef struct {
  uint32_t abi_version;                /* IODF_ABI_VERSION                                           */
  uint32_t in_c, in_h, in_w;           /* image shape; in_h, in_w divisible by 2^n_levels            */
  uint32_t n_levels;
  uint32_t max_batch;                  /* workspace is sized for this batch at create                */
  const iodf_level_desc* levels;       /* HOST                                                       */
  uint32_t plan;                       /* IODF_PLAN_LATENCY or IODF_PLAN_THROUGHPUT (else EINVAL)    */
} iodf_model_desc;

#define IODF_MAX_LEVELS 8

/* Shape of the latent. Per image, z is the concatenation, level 0 first, of every factored-out
 * block in [channel][row][col] order, followed by the last level's remaining channels. The prior
 * buffer holds, per image, d_fact values of mu followed by d_fact values of the log-scale index,
 * in the order of the factored-out blocks that have a prior head. */
typedef struct {
  uint64_t d;                              /* latent elements per image = in_c*in_h*in_w            */
  uint64_t d_fact;                         /* elements per image that have prior parameters         */
  uint32_t n_levels;
  uint32_t level_c[IODF_MAX_LEVELS], level_h[IODF_MAX_LEVELS], level_w[IODF_MAX_LEVELS];
  uint64_t z_off[IODF_MAX_LEVELS];         /* offset of the level's factored-out block in z         */
  uint64_t prior_off[IODF_MAX_LEVELS];     /* offset of the level's block in mu (and in ls)         */
  uint64_t z_final_off;                    /* offset of the final block                             */
  uint64_t macs_per_image;                 /* multiply-accumulates over the kept channels           */
} iodf_layout;

typedef struct iodf_model iodf_model;

/*
 * Validate `desc`, copy and repack weights and requant parameters to the device, size the
 * workspace for desc->max_batch. `weights`/`requant` are HOST arrays that may be freed afterwards.
 * `device` is a CUDA device ordinal; it is made current for the duration of the call.
 * Errors: EINVAL (null pointer; odd channel count; perm not a permutation; M0 outside
 * [2^30, 2^31); s outside [0, 31]; offsets beyond the blobs; layer shapes that do not chain),
 * EOVERFLOW, EVERSION, ENOMEM, ECUDA, EUNSUPPORTED. This build runs couplings of the form
 * conv3x3+ReLU+clip -> conv1x1+ReLU+clip -> conv3x3 with hidden activations inside the signed
 * 8-bit range and hidden widths up to 512 kept channels (above 256 the weights are streamed from
 * L2 for every tile instead of staying in shared memory), couplings with residual blocks (see
 * iodf_coupling_desc) at levels of at most 2048 pixels per image, and 3x3 prior heads.
 */
int iodf_create(const iodf_model_desc* desc, const int8_t* weights, size_t weights_count,
                const int32_t* requant, size_t requant_count, int device, iodf_model** out);

void iodf_destroy(iodf_model* m);

int iodf_get_layout(const iodf_model* m, iodf_layout* out);

/*
 * Encode, z = f(x) (Sec. 3: the flow is the composition of the levels' additive couplings, Eq. 2,
 * with the coupling networks evaluated in integers, Sec. 4.1; App. B.1 for the level structure):
 * x_u8 DEV uint8 [B][in_c][in_h][in_w]  ->  z DEV int32 [B][d] and, if `prior` is not NULL, prior
 * DEV int32 [B][2][d_fact] (the (mu, s) of Sec. 3's discretised logistic prior for every
 * factored-out element). 1 <= B <= max_batch. Pointers must be 16-byte aligned. Enqueues one
 * kernel per level on `cuda_stream`; allocates nothing; the caller owns all three buffers.
 * Errors: IODF_EINVAL (null or misaligned pointer, B out of range), IODF_ECUDA (launch failure).
 */
int iodf_forward(iodf_model* m, const uint8_t* x_u8, int B, int32_t* z, int32_t* prior, void* cuda_stream);

/*
 * Decode, x = f^-1(z) (Eq. 2 inverted: x_b = z_b - round(t(z_a)), levels and couplings in reverse
 * order, Sec. 3): z DEV int32 [B][d] -> x_u8 DEV uint8 [B][in_c][in_h][in_w] (the low 8 bits of each
 * recovered value). If `prior` is not NULL the same prior parameters as iodf_forward are written.
 * If `out_of_range_count` (DEV uint32) is not NULL, the number of recovered values outside 0..255
 * is ADDED to it (the caller zeroes it); this can only be non-zero for a z that no image encodes to.
 */
int iodf_inverse(iodf_model* m, const int32_t* z, int B, uint8_t* x_u8, int32_t* prior,
                 uint32_t* out_of_range_count, void* cuda_stream);

/*
 * Level-stepped decode, for a decompressor that alternates entropy decoding and flow inversion
 * (the multi-scale architecture of Sec. 5 / App. B.1: the prior of a level's factored-out block is
 * conditioned on the channels that the level keeps, which a decoder only knows once every deeper
 * level has been inverted; App. A decodes symbols with those parameters). Call order, for
 * level = n_levels-1 down to 0:
 *   IODF_LEVEL_PRIOR      prior parameters of the level's factored-out block (mu at
 *                         prior[b][0][prior_off[level] ..], log-scale index at prior[b][1][..]) from the
 *                         level's kept channels: z's final block for the deepest level, otherwise what
 *                         the IODF_LEVEL_COUPLINGS call of level+1 left in the model's workspace. No
 *                         other part of z is read, nothing else is written. Levels without a prior
 *                         head return IODF_EINVAL (their block has a fixed prior).
 *   (the caller entropy-decodes the level's block z[b][z_off[level] ..] with those parameters)
 *   IODF_LEVEL_COUPLINGS  merges the kept channels with the level's block of z, inverts the level's
 *                         couplings and the squeeze; the result is the kept input of level-1 (model
 *                         workspace) or, for level 0, x_u8 (and out_of_range_count, as iodf_inverse).
 *                         Reads only z's block of this level (and the final block at the deepest level).
 * z, prior, x_u8: DEV, full-size buffers with the layouts of iodf_forward; x_u8 is used at level 0
 * only and prior by IODF_LEVEL_PRIOR only (either may be NULL otherwise). The sequence over all
 * levels gives bit for bit what iodf_inverse gives. One sequence per model at a time.
 */
#define IODF_LEVEL_PRIOR 1
#define IODF_LEVEL_COUPLINGS 2
int iodf_inverse_level(iodf_model* m, int level, int phase, const int32_t* z, int B, uint8_t* x_u8, int32_t* prior,
                       uint32_t* out_of_range_count, void* cuda_stream);

/*
 * Patch-based coding of one high-resolution image (Sec. 5.3: a large image is cut into patches
 * of the training resolution, so one image already is a large batch). image_u8 is DEV
 * uint8 [in_c][H][W] with H, W multiples of in_h, in_w; patch b = (b / (W/in_w), b % (W/in_w)) in
 * row-major order is image b of a batch of B = (H/in_h)*(W/in_w) <= max_batch images. The cut is an
 * index map of the first level's load (encode) and last store (decode): no patch batch is
 * materialised. z is [B][d] and prior [B][2][d_fact] exactly as for iodf_forward on that batch.
 * Errors: IODF_EINVAL if H or W is not a multiple of the patch size or B exceeds max_batch.
 */
int iodf_forward_patches(iodf_model* m, const uint8_t* image_u8, int H, int W, int32_t* z, int32_t* prior,
                         void* cuda_stream);
int iodf_inverse_patches(iodf_model* m, const int32_t* z, int H, int W, uint8_t* image_u8, int32_t* prior,
                         uint32_t* out_of_range_count, void* cuda_stream);

/*
 * Entropy coding of the latents on the GPU (Sec. 3: factorised discrete logistic prior; App. A:
 * range-ANS; Sec. 5.3 codes on the CPU and names a GPU coder as future work).
 *
 * The prior's integer form is given by the caller (HOST arrays, copied):
 *   sigmoid_table[u + umax], u in [-umax, umax], umax <= 8192: a non-decreasing table of
 *     M' sigma(u / 64), M' = 2^16 - 4097, entries <= M';
 *   inv_scale[ls] = 2^21 / s_ls, in [1, 2^30), for scale index ls in [0, n_scales), n_scales <= 1024
 *     (the prior head's log-scale index);
 *   final_ls: the fixed scale index (with mu = 0) of blocks that have no prior head, the final block
 *     among them.
 * An element with prior (mu, ls) is coded as the symbol k = clamp(z - mu, -2048, 2048) + 2048 with
 *   Cum(k) = k + sigmoid_table[clamp(floor((2 (k - 2048) - 1) inv_scale[ls] / 2^16), -umax, umax) + umax],
 *   Cum(0) = 0, Cum(4097) = 2^16; k = 0 and k = 4096 are escapes followed by the 32 bits of z.
 * rANS: total mass M = 2^16, 32-bit state kept in [2^16, 2^32), 16-bit words; App. A's update
 * X' = floor(X / F) M + C + X mod F and its inverse.
 *
 * Container. Per image the coded blocks are every factored-out block in z order and then the final
 * block (a decoder needs a block's symbols before it can compute the next block's prior). Block q
 * of n elements is cut into ceil(n / elems_per_stream) streams; stream j holds elements j, j + ns, ...
 * words is DEV uint16 [B][n_streams][words_per_stream] and counts DEV uint32 [B][n_streams]; stream s
 * of image b occupies words[b][s][0 .. counts[b][s]) (emitted words, then the final state, low half
 * first); the compressed size of an image is 2 * sum of its counts bytes. iodf_codec_get_layout gives
 * the numbers. words_per_stream = 3 * elems_per_stream + 2 is the worst case.
 *
 * iodf_rans_encode codes every block of z [B][d] with prior [B][2][d_fact] (as written by
 * iodf_forward). iodf_rans_decode_block decodes one block of every image into z (the rest of z is
 * untouched); with iodf_inverse_level the decode order is: final block, then for level = deepest
 * .. 0: IODF_LEVEL_PRIOR, iodf_rans_decode_block(block of that level), IODF_LEVEL_COUPLINGS.
 * Both enqueue one kernel on `cuda_stream` and allocate nothing. A scale index outside
 * [0, n_scales) or a stream whose words do not end where they should is counted on the device and
 * reported by iodf_codec_check (IODF_EDATA), never dereferenced.
 */
typedef struct {
  uint32_t abi_version;              /* IODF_ABI_VERSION                                             */
  const uint16_t* sigmoid_table;     /* HOST, 2 * umax + 1 entries                                   */
  uint32_t umax;
  const uint32_t* inv_scale;         /* HOST, n_scales entries                                       */
  uint32_t n_scales;
  int32_t final_ls;
  uint32_t elems_per_stream;
} iodf_codec_desc;

typedef struct {
  uint32_t n_blocks;                                  /* coded blocks per image                      */
  uint32_t n_streams;                                 /* streams per image                           */
  uint32_t words_per_stream;                          /* container stride, in 16-bit words           */
  int32_t block_level[IODF_MAX_LEVELS + 1];           /* flow level of the block, -1: final block    */
  uint64_t block_z_off[IODF_MAX_LEVELS + 1];
  uint64_t block_elems[IODF_MAX_LEVELS + 1];
  uint32_t block_first_stream[IODF_MAX_LEVELS + 1];
  uint32_t block_streams[IODF_MAX_LEVELS + 1];
} iodf_codec_layout;

typedef struct iodf_codec iodf_codec;

int iodf_codec_create(const iodf_model* m, const iodf_codec_desc* desc, iodf_codec** out);
void iodf_codec_destroy(iodf_codec* c);
int iodf_codec_get_layout(const iodf_codec* c, iodf_codec_layout* out);
int iodf_rans_encode(iodf_codec* c, const int32_t* z, const int32_t* prior, int B, uint16_t* words, uint32_t* counts,
                     void* cuda_stream);
int iodf_rans_decode_block(iodf_codec* c, int block, const uint16_t* words, const uint32_t* counts,
                           const int32_t* prior, int B, int32_t* z, void* cuda_stream);
/*
 * Compact byte stream of a batch (what a file or a network message would hold; little endian):
 *   uint32 offset[B + 1]   byte offset of image b's record from the start of the payload;
 *                          offset[B] = payload bytes
 *   payload, per image:    uint16 count[n_streams], then the words of stream 0, 1, ... back to back
 * iodf_rans_pack writes it from a container (packed: DEV, 4-byte aligned, at least
 * iodf_rans_packed_capacity(c, B) bytes; the total is 4 (B + 1) + offset[B]); iodf_rans_unpack
 * restores the container from packed_bytes bytes, checking every record against the payload size
 * and its own counts (a bad record gets zero counts and is reported by iodf_codec_check). Both need
 * words_per_stream <= 65535 (IODF_EINVAL otherwise), at most 8192 streams per image and a byte stream
 * below 4 GiB (IODF_EUNSUPPORTED otherwise).
 */
size_t iodf_rans_packed_capacity(const iodf_codec* c, int B);
int iodf_rans_pack(iodf_codec* c, const uint16_t* words, const uint32_t* counts, int B, uint8_t* packed,
                   void* cuda_stream);
int iodf_rans_unpack(iodf_codec* c, const uint8_t* packed, size_t packed_bytes, int B, uint16_t* words,
                     uint32_t* counts, void* cuda_stream);

/*
 * Whole compressor and decompressor for HOST buffers (pinned memory recommended): images in, compact
 * byte stream out, and back. The latents and prior parameters stay on the device. The first call
 * allocates the codec's staging buffers for the model's max_batch (do it before any stream capture).
 * iodf_compress_host synchronises the stream (the size of the byte stream is data dependent) and
 * returns it in *out_bytes; IODF_ELIMIT if out_capacity is too small (*out_bytes then says how much
 * is needed). iodf_decompress_host enqueues everything and returns; x_u8_host is valid after the
 * stream has been synchronised, and iodf_codec_check / iodf_check report damaged input.
 */
int iodf_compress_host(iodf_model* m, iodf_codec* c, const uint8_t* x_u8_host, int B, uint8_t* out_host,
                       size_t out_capacity, size_t* out_bytes, void* cuda_stream);
int iodf_decompress_host(iodf_model* m, iodf_codec* c, const uint8_t* in_host, size_t in_bytes, int B,
                         uint8_t* x_u8_host, void* cuda_stream);

/* Synchronise the stream; IODF_EDATA if any stream was flagged since the last check (their number
 * in *bad_streams, HOST, may be NULL). */
int iodf_codec_check(iodf_codec* c, void* cuda_stream, uint32_t* bad_streams);

/*
 * The same two operations for HOST buffers (pinned memory recommended): inputs are copied to a
 * device staging area owned by the model, the flow runs, and the results are copied back, all
 * enqueued on `cuda_stream`; the host buffers are valid once the stream has been synchronised.
 */
int iodf_forward_host(iodf_model* m, const uint8_t* x_u8_host, int B, int32_t* z_host, int32_t* prior_host,
                      void* cuda_stream);
int iodf_inverse_host(iodf_model* m, const int32_t* z_host, int B, uint8_t* x_u8_host, void* cuda_stream);

/*
 * Synchronise `cuda_stream` and report the device status word: IODF_OK, IODF_ETIMEOUT if a
 * bounded wait inside a kernel gave up (the outputs of that call are then undefined), or
 * IODF_ECUDA. Clears the status word.
 */
int iodf_check(iodf_model* m, void* cuda_stream);

/*
 * Profiling variants: the same work as iodf_forward / iodf_inverse with a CUDA event recorded on
 * `cuda_stream` before and after each level's kernel. They synchronise the stream before returning
 * and write the device time of each level's kernel, in milliseconds, to level_ms[0 .. n_levels)
 * (HOST; level 0 is the finest level in both directions).
 */
int iodf_forward_timed(iodf_model* m, const uint8_t* x_u8, int B, int32_t* z, int32_t* prior, void* cuda_stream,
                       float* level_ms);
int iodf_inverse_timed(iodf_model* m, const int32_t* z, int B, uint8_t* x_u8, int32_t* prior,
                       uint32_t* out_of_range_count, void* cuda_stream, float* level_ms);

/*
 * Encode without touching any allocator (the paper has no counterpart; this exists for deployment).
 *
 * iodf_forward hands the kept channels from one level's kernel to the next through a workspace
 * that iodf_create sized with cudaMalloc for the model's max_batch. Some callers cannot have that:
 * a plug-in inside a host process that owns the device memory pool and forbids allocation, a
 * service whose model object was created for a small max_batch and which later sees a larger
 * batch at a point where allocating is not allowed (inside a latency-critical loop, or after the
 * rest of the device memory has been handed out). For them this entry point does the same encode,
 * with identical results, but keeps the inter-level data in a fixed array that is part of the
 * library image itself: IODF_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the
 * library, held until the process exits. It calls no allocation or free routine of any kind.
 *
 * Limits and rules
 *   - B is NOT limited by the model's max_batch but by the array: the call needs
 *     B * iodf_static_scratch_bytes_per_image(m) bytes and returns IODF_ELIMIT if that exceeds
 *     IODF_STATIC_SCRATCH_BYTES (nothing is launched).
 *   - The first call on a device looks up the array's device address (once per device, with the
 *     model's device made current for the lookup). Make that first call before any stream capture.
 *   - All calls, for all models on the device, share the one array; it keeps whatever the last
 *     call left in it. Nothing in it needs to start at zero (every level writes its part before the
 *     next level reads it), but two calls that overlap on the GPU (different streams, or this
 *     entry point from two threads without ordering) race on it. Serialise them on one stream.
 *   - x_u8, z, prior: DEV, as for iodf_forward.
 */
#define IODF_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)
int iodf_forward_static(iodf_model* m, const uint8_t* x_u8, int B, int32_t* z, int32_t* prior, void* cuda_stream);
/* Bytes of the fixed array one image needs for this model (0 for a single-level model). */
size_t iodf_static_scratch_bytes_per_image(const iodf_model* m);

/*
 * Self-test of the failure path (the paper has no counterpart). Every device-side wait of the
 * library is bounded: when its tries run out it sets the model's status word and the kernel drains
 * and returns, which iodf_check reports as IODF_ETIMEOUT. This call enqueues a one-warp kernel that
 * runs that same wait, with `tries` (1..100) suspended tries of up to 100 us each, on a barrier that
 * nothing arrives on, so that the path can be exercised without a fault: afterwards iodf_check
 * returns IODF_ETIMEOUT once, then IODF_OK, and the model works as before.
 */
int iodf_selftest_timeout(iodf_model* m, uint32_t tries, void* cuda_stream);

/*
 * The tensor roofline's denominator, measured (the paper has no counterpart; Sec. 4.1's point is
 * that the 8-bit multiply-accumulates dominate). Enqueues one kernel in which one CTA per SM issues
 * mma_groups * 8 tcgen05.mma kind::i8 instructions of shape 128 x 256 x 32 (int8 x int8 -> int32 in
 * tensor memory) from operands resident in shared memory, and nothing else. *ops_out (HOST, may be
 * NULL) receives the int8 OPs (2 per multiply-accumulate) of the launch; the caller times the
 * launch with events on `cuda_stream`. mma_groups in [1, 2^22]; m only supplies the device and
 * the status word of the kernel's bounded wait (check with iodf_check).
 */
int iodf_int8_mma_peak(iodf_model* m, uint32_t mma_groups, void* cuda_stream, unsigned long long* ops_out);

/* Name of the kernel template that runs level `level` of this model (for profiles and reports): the
 * library picks one per level when the model is created. "" for a bad argument. */
const char* iodf_level_kernel_name(const iodf_model* m, int level);

/* Images that one CTA of level `level`'s launch holds under the model's plan (1 where an image takes a
 * CTA, or a band of a cluster, of its own); a launch of B images has ceil(B / that) CTAs per band.
 * IODF_EINVAL for a bad argument. */
int iodf_level_images_per_cta(const iodf_model* m, int level);

/* Number of kernel launches one iodf_forward / iodf_inverse call enqueues. */
int iodf_launches_per_call(const iodf_model* m, int inverse);

const char* iodf_strerror(int status);
int iodf_last_cuda_error(const iodf_model* m); /* the cudaError_t behind the last IODF_ECUDA          */

#ifdef __cplusplus
}
#endif
#endif /* IODF_H_ */
