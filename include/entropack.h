/*
 * entropack.h -- C ABI of the B200-native EntroPack weight codec.
 *
 * EntroPack (arxiv 2609.34185) stores a weight matrix W[R][C] (C divisible by 8) as tiled,
 * 32-way interleaved rANS streams of E8 lattice-coordinate fields under a coset-conditioned
 * probability model, and reconstructs W-hat = snap_tau(sigma_r * p) on the GPU in one fused pass.
 *
 * Two halves:
 *   host  : ep_encode() and friends build the stored representation ("blob") on the CPU
 *           (paper Sec. 3.2-3.6, Algorithm 1, Eq. 13, Eq. 17).
 *   device: ep_decode_tensor() / ep_decode_batch() enqueue the fused sm_100a decode kernel
 *           (paper Sec. 3.7, Eq. 18, Eq. 5, Eq. 19).  There is no CPU decode path.
 *
 * Conventions
 *   - every function returns 0 (EP_OK) or a negative ep_status; no exceptions cross the ABI;
 *   - "host" pointers are ordinary memory, "device" pointers are CUDA global memory of the
 *     current device; the library never allocates or frees device memory and never
 *     synchronises inside a decode call: work is enqueued on the given stream;
 *   - `stream` arguments are cudaStream_t handles passed as void* (NULL = default stream);
 *   - all multi-byte stream fields are little-endian.
 *
 * Stored representation (all of it counts toward the stored rate of Eq. 1):
 *   [header 64 B]   magic "EPK1", u16 version=1, u8 b, u8 J=32, u32 R, u32 C, u32 V, u32 n_tiles,
 *                   f32 s (informational), i16 coord_min, i16 coord_max, u32 byte offsets of the four
 *                   sections below, u64 total bytes, u32 total payload words, u32 zero
 *   [tables]        i32 min[17], u32 K[17], then u16 freq[K_t] for t = 0..16, padded to 4 bytes.
 *                   t = 0 is the coset table; field k (1..7 = z_k, 8 = m) under coset c is
 *                   t = 1 + 8c + (k-1).  Frequencies of a non-empty table sum to 2^b.
 *   [row scales]    R x f32
 *   [tile index]    n_tiles x { u32 state[32], u32 word_offset }, then u32 final boundary offset
 *                   (132 bytes per tile + 4, as in the paper's tile-overhead table)
 *   [payload]       16-bit words of all tiles, concatenated, no padding
 * Tile t holds vectors [t*V, min((t+1)*V, R*C/8)) of the row-major sequence of 8-weight blocks.
 * Inside a tile, vector i uses rANS state i mod 32; decoding proceeds by groups of 32 vectors,
 * within a group by field (coset first, then z1..z7, m), within a field by lane 0..31; after its
 * symbol a lane whose state is below 2^15 takes the next payload word.
 */
#ifndef ENTROPACK_H
#define ENTROPACK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define EP_NUM_TABLES 17
#define EP_MAX_BATCH 16

typedef enum {
    EP_OK = 0,
    EP_ERR_BAD_ARG = -1,     /* NULL pointer, C % 8 != 0, size out of range, misaligned output */
    EP_ERR_BAD_STREAM = -2,  /* blob fails structural validation, or the decoder found an inconsistency */
    EP_ERR_UNSUPPORTED = -3, /* valid request this build cannot serve (e.g. offsets beyond 32 bits) */
    EP_ERR_CUDA = -4,        /* a CUDA runtime call failed */
    EP_ERR_NOMEM = -6,       /* host allocation failed */
    EP_ERR_SCRATCH = -7,     /* scratch buffer missing, misaligned or too small */
    EP_ERR_STATIC_LIMIT = -8 /* ep_decode_tensor_static: the stream's tables exceed the built-in area */
} ep_status;

/* Output element types of the decoder: snap_tau of Eq. 19. */
typedef enum {
    EP_BF16 = 0,        /* round to nearest even */
    EP_FP16 = 1,        /* round to nearest even, saturating to +-65504 */
    EP_FP8_E4M3 = 2,    /* E4M3FN, round to nearest even incl. subnormals, saturating to +-448 */
    EP_INT8 = 3,        /* round to nearest even integer, saturating to [-128, 127] */
    EP_FP32 = 4,        /* the fp32 product itself */
    EP_FP8_E5M2 = 5,    /* E5M2, round to nearest even incl. subnormals, saturating to +-57344 */
    EP_UINT8 = 6,       /* round to nearest even integer, saturating to [0, 255] (for weights that were
                           shifted into the unsigned range before compression) */
    EP_FIELDS_I32 = 16  /* verification mode: the nine decoded fields (c, z1..z7, m) of Eq. 4 as
                           int32[R*C/8][9]; row scales are not read */
} ep_dtype;

/* Encoder settings; ep_encode_opts_default() fills in the paper's values
 * (App. "Scale-search settings", App. "Tile layout and storage"). */
typedef struct {
    double bracket_lo, bracket_hi; /* geometric search bracket for s: [1e-3, 8] */
    int32_t search_steps;          /* I_s = 12 bisection steps */
    uint32_t sample_vectors;       /* nominal row-sample budget: 2^18 eight-vectors */
    uint32_t tile_vectors;         /* V; 0 = max(32, floor(S/9)) with S from the target rate */
    int32_t b_start;               /* 0 = 11 for targets <= 7 bpp, 12 above */
    int32_t b_max;                 /* 15 */
    double retained_bits;          /* constant of Eq. 10 (bits assumed to stay in each state): 16 */
    int32_t polish_steps;          /* corrections of s from the full-tensor estimate after Algorithm 1 (an
                                      addition to the paper's procedure; 0 = the literal Algorithm 1): 3 */
    double polish_retained_bits;   /* bits per state taken as retained in those corrections: 8 (states end up
                                      spread over [2^15, 2^31), so about 8 bits each stay out of the payload) */
    int32_t threads;               /* host worker threads; 0 = all hardware threads */
    int32_t rdo_candidates;        /* K of the per-row rate-distortion refinement (Sec. 3.5, Alg. 2): candidate
                                      scales rho_k * s per row, rho in [0.70, 1.45]; 1 = off (the paper's default).
                                      Host encoder only */
    int32_t rdo_sweeps;            /* T allocation / model-update sweeps: 1 */
} ep_encode_opts;

/* What the encoder decided; filled by ep_blob_report(). */
typedef struct {
    double s;               /* selected search scale */
    double stored_bpp;      /* Eq. 1: 8 * bytes / (R*C) */
    double est_bpp_sample;  /* Eq. 12 at the last evaluated candidate of the chosen precision */
    double cce_bits;        /* Eq. 8 on the final full-tensor tables */
    uint64_t bytes;
    uint32_t sample_rows;
    int32_t b;
} ep_encode_report;

/* Host-side description of a blob: a copy of its header and table directory.  Obtained once from
 * the host copy of the blob with ep_blob_info() and handed to the decode calls, which therefore
 * never read device memory on the host. */
typedef struct {
    uint32_t R, C, V, n_tiles;
    uint32_t b, J;
    int32_t coord_min, coord_max;     /* range of the integer coordinates z_1..z_8 over the tensor */
    float s;
    uint32_t off_tables, off_scales, off_tiles, off_payload;  /* byte offsets inside the blob */
    uint64_t total_bytes;
    uint64_t total_words;
    int32_t table_min[EP_NUM_TABLES];   /* alphabet offset of each table */
    uint32_t table_K[EP_NUM_TABLES];    /* stored entries of each table (0 = table never used) */
} ep_info;

typedef struct ep_blob ep_blob;   /* host-owned stored representation */

/* One tensor of a batched decode.  All pointers except `info` are device pointers. */
typedef struct {
    const ep_info *info;        /* host */
    const void *d_stream;       /* device: the blob, or at least its header, table and payload sections,
                                   at their blob offsets; 4-byte aligned */
    const void *d_tile_index;   /* device: the tile-index section (132*n_tiles + 4 bytes); 4-byte aligned */
    const float *d_row_scales;  /* device: R fp32 row scales (the blob's, or the caller's own) */
    int32_t out_dtype;          /* ep_dtype */
    void *d_out;                /* device: R*C elements of out_dtype, row-major; 16-byte aligned (8 bytes are
                                   enough for the one-byte types, 4 for EP_FIELDS_I32) */
    void *d_scratch;            /* device: ep_decode_scratch_bytes(info) bytes, 256-byte aligned; may be
                                   NULL when that size is 0 */
    size_t scratch_bytes;
    uint32_t tile_begin;        /* a range of tiles to decode, for a caller that owns a shard of the tensor */
    uint32_t tile_count;        /* (both 0 = the whole tensor); see ep_decode_tiles */
    const void *d_tables;       /* device: lookup tables of this stream as ep_prepare_tables() left them
                                   (ep_decode_tables_bytes(info) bytes, 256-byte aligned), or NULL: the decode
                                   then derives them from the stream's frequency tables on every call.  With
                                   prepared tables d_scratch is not needed */
} ep_decode_job;

/* ---- host encoder ------------------------------------------------------------------------- */

/* Paper defaults for every field of *opts. */
void ep_encode_opts_default(ep_encode_opts *opts);

/* Compress W (host, row-major R x C fp32, C % 8 == 0, R*C/8 < 2^32) to about target_bpp stored
 * bits per weight: row RMS normalisation, E8 nearest-point quantisation, sampled storage estimate,
 * geometric scale search with precision escalation (Algorithm 1), row-scale refit (Eq. 13), final
 * tables and tiled rANS encoding (Eq. 17).  opts may be NULL.  On success *out owns the blob;
 * release it with ep_blob_free().  W is only read. */
int ep_encode(const float *W, uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts *opts,
              ep_blob **out);

/* Encode given fields directly (final tables + tile coding only; Sec. 3.6).  fields is host
 * int32[R*C/8][9] = (c, z1..z7, m) per block, row_scales host f32[R].  For tools and tests. */
int ep_pack_fields(const int32_t *fields, uint32_t R, uint32_t C, int32_t b, uint32_t V,
                   const float *row_scales, float s_info, int32_t threads, ep_blob **out);

/* The same encoder with the heavy steps on the GPU (row RMS, E8 quantisation and field histograms, Eq. 13,
 * tile coding); the search itself and the table arithmetic stay on the host, so the result is byte for
 * byte the blob ep_encode produces for the same W and options.  d_W is a device copy of W (16-byte
 * aligned), d_workspace a 256-byte aligned device buffer of ep_encode_device_workspace_bytes() bytes
 * (about 54 bytes per 8-weight block).  The call enqueues on `stream` and synchronises it several times;
 * it returns the finished host blob.  EP_ERR_UNSUPPORTED (use ep_encode instead) if a lattice coordinate
 * exceeds +-4095 or the tables hold more than 40960 symbols in total.
 * The blob of this call lives in page-locked host memory (the device copies the payload straight into it,
 * and a later upload of the blob runs at full bus speed).  Page-locking costs milliseconds, so ep_blob_free
 * keeps the buffer of the most recently freed such blob (one per process at most, the larger one when two
 * compete) for the next call whose blob fits; a model converted tensor by tensor allocates once or twice.
 * A second page-locked buffer of 0.5 MB (the histograms of the counting passes) is kept the same way. */
size_t ep_encode_device_workspace_bytes(uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts *opts);
int ep_encode_device(const float *d_W, uint32_t R, uint32_t C, double target_bpp, const ep_encode_opts *opts,
                     void *d_workspace, size_t workspace_bytes, void *stream, ep_blob **out);

const void *ep_blob_data(const ep_blob *blob);   /* host pointer valid until ep_blob_free */
size_t ep_blob_bytes(const ep_blob *blob);       /* B_stored of Eq. 1 */
int ep_blob_report(const ep_blob *blob, ep_encode_report *out);
void ep_blob_free(ep_blob *blob);

/* Parse header and table directory of a host copy of a blob (n bytes): the "tensor layout" and "frequency tables,
 * alphabet offsets" parts of the stored representation (Sec. 3.6, paragraph on the stored representation;
 * App. "Tile layout and storage").  EP_ERR_BAD_STREAM if the bytes are not a blob of this format. */
int ep_blob_info(const void *blob, size_t n, ep_info *out);

/* Full structural check of a host copy of a blob against what the stored representation must satisfy (Sec. 3.6;
 * App. "Tile layout and storage", "State normalisation"): sizes and offsets consistent and monotone,
 * frequencies of every used table sum to 2^b (Sec. 3.3), states inside [2^15, 2^31).  A blob that passes can
 * be given to the decoder without risk of out-of-range accesses. */
int ep_validate(const void *blob, size_t n);

/* ---- device decoder ----------------------------------------------------------------------- */

/* Scratch bytes the decoder needs for this tensor: 0 when the symbol lookup tables fit shared
 * memory (b <= 11 and coordinate range <= 1024, no single-symbol table at b = 11), else room
 * for 17 tables of 2^b four-byte entries. */
size_t ep_decode_scratch_bytes(const ep_info *info);

/* The decoder's lookup tables (App. "Tiled RANS implementation": the low b bits of a state select symbol and
 * interval) depend on the stream's frequency tables only, and a weight is decoded on every forward call
 * (Sec. "Reconstruction cost and tile overhead").  A caller that keeps a stream resident can therefore have
 * them derived once: ep_decode_tables_bytes() is the size of the table image for this stream (128 KB when
 * the tables fit shared memory, else 17 tables of 2^b four-byte entries), ep_prepare_tables() enqueues one
 * small launch on `stream` that fills d_tables (device, 256-byte aligned) from the device copy of the blob,
 * and every later decode of that stream that passes d_tables in its ep_decode_job copies (or reads) the image
 * instead of rebuilding it.  The image is opaque and valid for this library version, this stream and any
 * tile range of it.  Errors: EP_ERR_SCRATCH for a missing, misaligned or short buffer. */
size_t ep_decode_tables_bytes(const ep_info *info);
int ep_prepare_tables(const ep_info *info, const void *d_stream, void *d_tables, size_t tables_bytes, void *stream);

/* Tiles the decode kernel works on at a time per SM (48: 24 warps, two tiles each); times the SM count this
 * is the `decode_slots` argument of ep_suggest_tile_vectors (App. "Tile layout and storage": tile size trades
 * storage against parallelism). */
uint32_t ep_decode_tiles_per_sm(void);

/* Fused decode of one tensor (Sec. 3.7): rANS symbol decode (Eq. 18) -> inverse field transform
 * (Eq. 5) -> multiply by the fp32 row scale -> snap to out_dtype (Eq. 19) -> store.  Enqueues on
 * `stream` and returns; see ep_decode_job for the pointer arguments.  The first decode call per output
 * type on a device also sets an attribute of the kernel (its shared-memory size); after that a call does
 * nothing but enqueue its launches, so it can be recorded in a stream capture and replayed as a CUDA graph. */
int ep_decode_tensor(const ep_info *info, const void *d_stream, const void *d_tile_index,
                     const float *d_row_scales, int32_t out_dtype, void *d_out, void *d_scratch,
                     size_t scratch_bytes, void *stream);

/* Tiles are independently decodable (Sec. 3.6): this call decodes tiles [tile_begin, tile_begin + tile_count)
 * only, i.e. blocks [tile_begin * V, min((tile_begin + tile_count) * V, R*C/8)) of the row-major block
 * sequence, and writes nothing else.  d_out is still the address of element (0, 0) of the full tensor: a
 * caller that holds only its shard passes shard_base - first_block * 8 * sizeof(element) (which must keep
 * d_out's alignment; it is never dereferenced outside the shard).  d_row_scales is indexed by the tensor's row
 * numbers likewise.  tile_count >= 1, tile_begin + tile_count <= n_tiles, else EP_ERR_BAD_ARG.  With this,
 * ranks of a tensor-parallel job decode disjoint row ranges of one stream without any exchange. */
int ep_decode_tiles(const ep_info *info, const void *d_stream, const void *d_tile_index,
                    const float *d_row_scales, int32_t out_dtype, void *d_out, void *d_scratch,
                    size_t scratch_bytes, uint32_t tile_begin, uint32_t tile_count, void *stream);

/* The same decode (Sec. 3.7) for up to EP_MAX_BATCH tensors in one kernel launch: tiles are independently
 * decodable (Sec. 3.6), so the tiles of all tensors share one grid - the way the paper's per-layer use decodes the
 * weights of a block before its matrix products (Sec. "Reconstruction cost and tile overhead").  All jobs of a call
 * have the same out_dtype.  Jobs needing scratch get their lookup tables built by one extra launch first. */
int ep_decode_batch(const ep_decode_job *jobs, int32_t n_jobs, void *stream);

/* Largest probability precision b served by ep_decode_tensor_static: its built-in table area holds
 * 17 tables of 2^13 four-byte entries = 557 056 bytes of device memory per GPU that loads the library. */
#define EP_STATIC_MAX_B 13

/* (No counterpart in the paper: an integration aid of this library.)
 * Same decode as ep_decode_tensor, for callers that cannot hand over a scratch buffer because they
 * cannot allocate device memory at the point of the call: code running inside a host framework that owns
 * the allocator and passes in nothing but input and output buffers, or a serving loop in which a
 * cudaMalloc would stall the whole device.  Streams whose lookup tables do not fit shared memory
 * normally need ep_decode_scratch_bytes() of caller memory; here the tables are built in a fixed area
 * compiled into the library instead.  The call itself allocates and frees nothing.
 *   - Limit: b <= EP_STATIC_MAX_B.  A stream with larger b is refused with EP_ERR_STATIC_LIMIT (use
 *     ep_decode_tensor with your own scratch for those).  Streams that need no scratch are decoded
 *     exactly as by ep_decode_tensor.
 *   - The first call on each device looks up the device address of the built-in area (the device must be
 *     current); make that first call before any stream capture begins.
 *   - All calls on a device share the one area and it keeps whatever the previous call left there; each
 *     call rewrites every table it reads, so nothing has to be cleared, but two calls whose kernels
 *     overlap on the GPU (different streams, no ordering between them) race on it.  Serialise them. */
int ep_decode_tensor_static(const ep_info *info, const void *d_stream, const void *d_tile_index,
                            const float *d_row_scales, int32_t out_dtype, void *d_out, void *stream);

/* Decode fused into a matrix product, first slice (the paper leaves this as future work, Sec. "Limitations and
 * future work": its decoder materialises the dense tensor and the product reads it back; the right panel of the
 * reconstruction-cost experiment shows what that costs at small token counts).  Computes
 *     y[t, r] = sum_k x[t, k] * W^[r, k],   W^ = the stream decoded to BF16 (Eq. 18, Eq. 5, Eq. 19 with tau = BF16),
 * with BF16 products accumulated in fp32 by the tensor cores; W^ is never written to global memory.
 *   d_x   device, T x C bfloat16, row-major, 16-byte aligned (T tokens, 1 <= T <= 32)
 *   d_y   device, T x R float, row-major, 16-byte aligned; every element is written
 *   d_tables  device, the prepared lookup tables of the stream (ep_prepare_tables); required
 * The stream must be laid out for it: one tile per row (V = C / 8; ep_encode with tile_vectors = C / 8), C a multiple
 * of 256, b = 11 with tables that fit shared memory (ep_decode_scratch_bytes(info) == 0).  Anything else returns
 * EP_ERR_UNSUPPORTED; decode with ep_decode_tensor and multiply separately then.  Asynchronous on `stream`, allocates
 * nothing (it asks the driver for a tensor-map descriptor of x, a host-side call).  A wait inside the kernel that
 * does not end raises the integrity word below instead of hanging. */
int ep_decode_gemm(const ep_info *info, const void *d_stream, const void *d_tile_index, const float *d_row_scales,
                   const void *d_tables, const void *d_x, uint32_t T, float *d_y, void *stream);

/* Device-side integrity word (no counterpart in the paper; it uses the fact that the encoder of Eq. 17 starts
 * every state at 2^15, so a correct decode of Eq. 18 must end there).  The kernel ORs in a flag when a tile does
 * not end with every state at 2^15 and its word pointer at the next tile's offset (a damaged stream).  There is ONE
 * such word per device and process, shared by all streams and callers: the `stream` argument only says which
 * stream to wait for.  This call synchronises `stream`, returns EP_OK or EP_ERR_BAD_STREAM / EP_ERR_CUDA, and
 * clears the word.
 * For tests and debugging; not needed on the hot path.  The decode kernels take every address bound
 * from `info` (sizes, counts, offsets), never from the stream's contents: damaged tables, tile records
 * or payload give wrong weights and this flag, not an access outside the buffers `info` describes.
 * `info` itself must match the buffers (ep_blob_info / ep_validate on the host copy). */
int ep_last_device_status(void *stream);

/* ---- misc --------------------------------------------------------------------------------- */
const char *ep_strerror(int status);                  /* text of an ep_status value (library convention, not the paper's) */
uint32_t ep_default_tile_vectors(double target_bpp);  /* V from the paper's tile-size defaults */

/* Tile size for a decoder with `decode_slots` concurrent tile slots (ep_decode_tiles_per_sm() = 32 per SM for this library: 4736 on
 * a 148-SM B200): the largest V not above the paper's default for the target rate for which the tensor's
 * R*C/8 blocks split into a whole number of rounds of decode_slots tiles (the last round nearly full),
 * rounded up to a multiple of 32 vectors when that stays within the default.
 * Larger tiles amortise the 132 bytes of per-tile metadata, but a tensor with fewer tiles than slots
 * leaves SMs idle (App. "Tile layout and storage": tile size trades storage against parallelism).
 * Never below a quarter of the default rounded down to a multiple of 32 (small tensors); returns the default when decode_slots is 0. */
uint32_t ep_suggest_tile_vectors(uint32_t R, uint32_t C, double target_bpp, uint32_t decode_slots);

/* The same question for tensors that are decoded together by one ep_decode_batch launch (the blocks of a
 * transformer layer): one tile size for all of them, a multiple of 32 not above the paper's default, chosen
 * so that the rounds of all tensors (32 tiles per CTA and round) split over `decode_ctas` CTAs (the SM count:
 * 148 on a B200) with the shortest last round.  R[i] x C[i] are the n tensor shapes. */
uint32_t ep_suggest_tile_vectors_batch(const uint32_t *R, const uint32_t *C, uint32_t n, double target_bpp,
                                       uint32_t decode_ctas);
int ep_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ENTROPACK_H */
