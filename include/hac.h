/*
 * hac.h - C ABI of the HAC / sHAC compressed-domain product library for NVIDIA B200 (sm_100a).
 *
 * The formats and the product are those of Marino, Petrini, Malchiodi, Frasca, "Compact
 * representations of convolutional neural networks via weight pruning and quantization":
 *   HAC  (Sect. IV-B): the matrix as a column-order address map whose entries, zeros included,
 *        are replaced by Huffman code words; the bit string is stored in 32-bit words.
 *   sHAC (Sect. IV-C): the CSC vectors nz, ri, cb of the matrix with nz Huffman coded.
 *   Dot  (Algorithms 1-3): x^T W computed on the compressed representation, one output per
 *        column of W, for one input vector or a batch of them.
 *
 * Conventions
 *   - Every call returns an int status: HAC_OK (0) or a negative HAC_ERR_* code; nothing throws.
 *     hac_status_string() gives the text.  On error, outputs are left untouched unless stated.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global memory of the
 *     current device.  The library never allocates device memory: the caller provides the buffer a
 *     format is uploaded to, the inputs, the outputs and the workspace.  `cuda_stream` is a
 *     cudaStream_t passed as void* (NULL = the legacy default stream); device work is enqueued on
 *     it and the call returns without waiting, unless stated.
 *   - Handles are opaque, created by *_build, owned by the caller, released by *_free.  A handle
 *     may be used from one thread at a time.
 *   - Indices are 0-based (the paper counts from 1).  W is n x m: n inputs (rows), m outputs
 *     (columns).  b = 32 bits per memory word.
 */
#ifndef HAC_H_
#define HAC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HAC_OK                    0
#define HAC_ERR_INVALID_ARG      -1   /* null pointer, bad size, bad parameter                    */
#define HAC_ERR_ALLOC            -2   /* host allocation failed                                   */
#define HAC_ERR_NONFINITE_INPUT  -3   /* W holds NaN or Inf                                       */
#define HAC_ERR_K_TOO_LARGE      -4   /* more than HAC_MAX_SYMBOLS distinct values after sharing  */
#define HAC_ERR_CODE_TOO_LONG    -5   /* a Huffman code word longer than 32 bits                  */
#define HAC_ERR_OFFSET_OVERFLOW  -6   /* a size or offset does not fit its field                  */
#define HAC_ERR_NOT_UPLOADED     -7   /* device call on a format that was not uploaded            */
#define HAC_ERR_BUFFER_TOO_SMALL -8   /* caller's buffer or workspace too small                   */
#define HAC_ERR_CUDA             -9   /* a CUDA runtime call failed                               */
#define HAC_ERR_CORRUPT          -10  /* serialized data fails validation (*_deserialize, *_decode_host) */

#define HAC_MAX_SYMBOLS        4096   /* largest alphabet (distinct values, zero included)        */
#define HAC_MAX_SEG_SYMBOLS    1024   /* largest sub-segment length of the offset index           */

#define HAC_QUANT_NONE     0u   /* W already holds few distinct values                            */
#define HAC_QUANT_KMEANS   1u   /* CWS, Sect. III-C.1                                             */
#define HAC_QUANT_UNIFORM  2u   /* UQ,  Sect. III-C.3, grid over [min, max] of the non-null weights */
#define HAC_QUANT_GRID     3u   /* UQ as printed in Sect. III-C.3 with d = 0: w = delta * round(w / delta),
                                   delta tuned by bisection to leave at most k distinct values          */
#define HAC_QUANT_PWS      4u   /* PWS, Sect. III-C.2: k representatives at the i/(k-1) quantiles of the non-null
                                   weights; a weight between two of them goes to the upper one with probability
                                   (w - lo)/(hi - lo), drawn with SplitMix64 from `seed` and the weight's position */

typedef struct hac_format  hac_format;    /* HAC : stream, codebook, code lengths, offset index          */
typedef struct shac_format shac_format;   /* sHAC: stream of nz, ri, cb, codebook, lengths, offset index */

/* Build parameters (Sect. III-B, III-C).  Zero-initialise, then set what is needed. */
typedef struct hac_build_params {
    double   sparsity;      /* target fraction of zeros in [0,1); 0 = no pruning (Sect. III-B)          */
    uint32_t k;             /* number of shared values for the non-null weights (Sect. III-C)           */
    uint32_t quantizer;     /* HAC_QUANT_*                                                              */
    uint32_t kmeans_iters;  /* Lloyd iterations, run in full (no early stop)                            */
    uint32_t seg_symbols;   /* S: symbols per sub-segment of the offset index, 1..HAC_MAX_SEG_SYMBOLS;
                               0 = default: 64 for HAC; for sHAC about (entries of the fullest column)/64,
                               rounded up so that S * ri_bits / 32 is odd (reported by *_sizes)         */
    uint64_t seed;          /* seed of the k-means initialisation and of the draws of PWS               */
    uint32_t ri_bits;       /* sHAC: width of a stored row index, 16 or 32; 0 = 16 if n <= 65536 else 32
                               (the footnote of Sect. IV-A: ri needs only ceil(log n) bits)             */
    uint32_t reserved;      /* must be 0                                                                */
} hac_build_params;

/* Sizes of a built format.  "paper_bits" follows the paper's accounting (stream words, 6*k*b bits
 * for the two dictionaries kept as B-trees, and for sHAC ri and cb at b bits per entry); the
 * *_bytes fields are what this library really stores.  bound_bits is Corollary 1 (HAC) or
 * Corollary 2 (sHAC) evaluated at the format's own k and number of stored entries. */
typedef struct hac_size_report {
    int64_t n, m;               /* shape of W                                                     */
    int64_t nnz;                /* entries that survived pruning (stored entries of sHAC)         */
    int64_t symbols;            /* code words in the stream: n*m (HAC) or nnz (sHAC)              */
    int64_t stream_bits;        /* |HAC(W)| or |HAC(nz)|: sum of code word lengths                */
    int64_t stream_words;       /* N = ceil(stream_bits / 32)                                     */
    int64_t stream_bytes;       /* 4 * N                                                          */
    int64_t pad_bytes;          /* zero words appended after word N (alignment + over-read slack)  */
    int64_t codebook_bytes;     /* 4 * k_eff                                                      */
    int64_t code_len_bytes;     /* k_eff                                                          */
    int64_t ri_bytes;           /* sHAC: nnz * ri_bits / 8                                        */
    int64_t cb_bytes;           /* sHAC: 4 * (m + 1)                                              */
    int64_t offset_index_bytes; /* all arrays of the offset index                                 */
    int64_t total_bytes;        /* sum of the *_bytes fields above                                */
    int64_t paper_bits;         /* size by the paper's accounting                                 */
    double  bound_bits;         /* Corollary 1 / Corollary 2                                      */
    double  entropy;            /* source entropy H, bits per symbol                              */
    double  avg_code_len;       /* stream_bits / symbols                                          */
    uint32_t k_eff;             /* alphabet size                                                  */
    uint32_t max_code_len;
    uint32_t min_code_len;
    uint32_t seg_symbols;       /* S                                                              */
    uint32_t ri_bits;
    uint32_t units;             /* segments (warp work units) in the offset index                 */
} hac_size_report;

/* Borrowed host pointers to every array of a format; valid until the handle is freed.
 * Symbol id = rank of the value in `codebook` (ascending).  `stream` has stream_words data
 * words followed by stream_pad_words zero words.  Offset index: see hac_build. */
typedef struct hac_host_view {
    int64_t n, m;
    uint32_t k_eff, seg_symbols;
    const float*    codebook;      /* [k_eff] shared values, ascending                            */
    const uint8_t*  code_len;      /* [k_eff] code word length of each symbol                     */
    const uint32_t* codes;         /* [k_eff] canonical code word of each symbol (right aligned)  */
    const int64_t*  counts;        /* [k_eff] occurrences of each symbol                          */
    const uint32_t* stream;        /* [stream_words + stream_pad_words]                           */
    int64_t stream_bits, stream_words, stream_pad_words;
    uint32_t units;                /* U                                                           */
    uint32_t segs_per_col;         /* HAC: G; sHAC: 0                                             */
    const uint64_t* seg_bit_off;   /* [U]                                                         */
    const uint16_t* sub_bits;      /* [U * 32]                                                    */
} hac_host_view;

typedef struct shac_host_view {
    hac_host_view   base;          /* stream etc. of nz                                           */
    int64_t nnz;
    uint32_t ri_bits;
    const void*     ri;            /* [nnz] uint16_t or uint32_t row indices                      */
    const uint32_t* cb;            /* [m + 1] cb[j] = stored entries in columns before j          */
    const uint32_t* seg_first;     /* [m + 1] segments in columns before j                        */
    const uint32_t* seg_col;       /* [U] column of each segment                                  */
} shac_host_view;

/* ---------------------------------------------------------------------------------------------
 * hac_build / shac_build - Sect. III-B (pruning), III-C.1 / III-C.3 (weight sharing), IV-B / IV-C
 * (formats).  Host only, synchronous.
 *   W      host, row-major n x m fp32 with leading dimension ldw >= m (elements); borrowed for the
 *          duration of the call.  NaN / Inf -> HAC_ERR_NONFINITE_INPUT.  -0.0 counts as 0.
 *   params see hac_build_params.
 *   out    receives the new handle.
 * Steps:
 *   1. Pruning (Sect. III-B): entries with |w| <= the floor(sparsity*n*m)-th smallest magnitude become 0.
 *   2. Weight sharing (Sect. III-C) of the others, taken in column-major order, by `quantizer`:
 *        HAC_QUANT_KMEANS   k-means (Lloyd, kmeans_iters updates, start drawn from `seed`);
 *        HAC_QUANT_UNIFORM  a uniform grid of k levels over [min, max];
 *        HAC_QUANT_GRID     the zero-anchored grid delta * round(w / delta); delta is found by 70 halvings
 *                           of [0, 4 max|w|]: a trial delta that leaves at most k distinct values becomes
 *                           the upper end, and the upper end is used;
 *        HAC_QUANT_PWS      probabilistic sharing between the two neighbouring i/(k-1) quantiles (the i-th
 *                           quantile is the order statistic floor(i (q-1)/(k-1)) of the q non-null weights;
 *                           weight p draws (SplitMix64(seed + (p+1) * 0x9E3779B97F4A7C15) >> 11) * 2^-53);
 *        HAC_QUANT_NONE     none.
 *      Weights with at most k distinct values are kept as they are.
 *   3. The distinct values, sorted ascending, form the codebook.
 *   4. A Huffman code over the symbol counts (HAC: every entry, zeros included; sHAC: stored entries
 *      only), made canonical.
 *   5. Code words concatenated column by column, most significant bit first, into 32-bit words.
 * Offset index (the column-offset vector suggested in the paper's conclusions, refined): each column
 * (HAC: its n entries; sHAC: its stored entries) is cut into sub-segments of S symbols, 32
 * consecutive sub-segments form a segment; seg_bit_off[u] is the bit where segment u starts and
 * sub_bits[u*32 + l] the bit length of its l-th sub-segment.  HAC numbers segments u = j*G + g with
 * G = ceil(ceil(n/S)/32); sHAC numbers them column after column and adds seg_first, seg_col.
 * ------------------------------------------------------------------------------------------- */
int hac_build (const float* W, int64_t n, int64_t m, int64_t ldw, const hac_build_params* params,
               hac_format** out);
int shac_build(const float* W, int64_t n, int64_t m, int64_t ldw, const hac_build_params* params,
               shac_format** out);

/* ---------------------------------------------------------------------------------------------
 * hac_build_unified - several matrices quantized at the same time with one k and coded with one dictionary
 * (the "unified" quantization of Sect. V-D: uCWS, uPWS, uUQ).  Host only.
 *   1. Every matrix is pruned on its own (step 1 of hac_build, the same sparsity for all).
 *   2. The non-null weights of all matrices, matrix after matrix in the order given and column-major inside
 *      each, go through the weight sharing of params->quantizer together: one set of at most k shared values.
 *   3. One codebook (the distinct shared values of all matrices, plus 0 when a HAC matrix has a null entry) and
 *      one Huffman code on the symbol counts of all the streams together.
 *   4. Every matrix is emitted with that code as a format of its own (out[i] is a hac_format* when
 *      layers[i].sparse == 0, a shac_format* when it is 1), to be used, serialized and freed like any other.
 *      Each keeps the whole shared codebook and code (a symbol that does not occur in it has count 0), so
 *      hac_sizes counts the dictionary once per matrix; as the paper counts a unified model the dictionary
 *      term 6 k b of paper_bits is paid once for all of them.
 * With one matrix the result equals hac_build / shac_build.  On error no handle is returned.
 * Errors as hac_build; HAC_ERR_INVALID_ARG also for n_layers outside [1, HAC_MAX_UNIFIED_LAYERS].
 * ------------------------------------------------------------------------------------------- */
#define HAC_MAX_UNIFIED_LAYERS 1024
typedef struct {
    const float* W;           /* host, row-major, borrowed for the call */
    int64_t      n, m, ldw;
    int32_t      sparse;      /* 0: HAC, 1: sHAC */
    int32_t      reserved;
} hac_unified_layer;
int hac_build_unified(const hac_unified_layer* layers, int n_layers, const hac_build_params* params, void** out);

/* Sizes (Corollaries 1 and 2 for bound_bits) and borrowed views of the built arrays. Host only. */
int hac_sizes  (const hac_format*  f, hac_size_report* out);
int shac_sizes (const shac_format* f, hac_size_report* out);
int hac_export (const hac_format*  f, hac_host_view*  out);
int shac_export(const shac_format* f, shac_host_view* out);

/* The pruned and quantized matrix the format encodes, written to a host buffer Wq (row-major n x m,
 * leading dimension ldq >= m), reconstructed on the host from the stream (lossless, Sect. IV-B). */
int hac_decode_host (const hac_format*  f, float* Wq, int64_t ldq);
int shac_decode_host(const shac_format* f, float* Wq, int64_t ldq);

/* ---------------------------------------------------------------------------------------------
 * A built format as one flat little-endian byte string (the formats are the stored artefact, Sect. IV):
 * *_serialize_bytes gives its length, *_serialize writes it into the caller's host buffer, and
 * *_deserialize makes a new handle from such a string (released with *_free like any other).  The
 * string holds what is stored (codebook, code lengths, counts, stream, offset index, ri, cb) and a
 * checksum; decoding tables and work lists are rebuilt on load.  *_deserialize trusts nothing: a string
 * that is truncated, altered, inconsistent with its own header, or whose code, offset index or CSC
 * vectors are not valid gives HAC_ERR_CORRUPT (a string of the other format: HAC_ERR_INVALID_ARG).
 * Host only.
 * ------------------------------------------------------------------------------------------- */
int hac_serialize_bytes (const hac_format*  f, size_t* out);
int shac_serialize_bytes(const shac_format* f, size_t* out);
int hac_serialize (const hac_format*  f, void* buf, size_t bytes);
int shac_serialize(const shac_format* f, void* buf, size_t bytes);
int hac_deserialize (const void* buf, size_t bytes, hac_format**  out);
int shac_deserialize(const void* buf, size_t bytes, shac_format** out);

/* ---------------------------------------------------------------------------------------------
 * Upload.  *_device_bytes gives the size of the device image of a format (all arrays the kernels
 * read, plus decoding tables derived from the code lengths).  *_upload copies that image into the
 * caller's device buffer `dev_buf` (256-byte aligned, at least *_device_bytes long) on `cuda_stream`
 * and records the pointers in the handle.  The buffer stays owned by the caller and must outlive
 * every dot call on the handle.  Uploading again (e.g. to another buffer) re-targets the handle.
 * ------------------------------------------------------------------------------------------- */
int hac_device_bytes (const hac_format*  f, size_t* out);
int shac_device_bytes(const shac_format* f, size_t* out);
int hac_upload (hac_format*  f, void* dev_buf, size_t dev_bytes, void* cuda_stream);
int shac_upload(shac_format* f, void* dev_buf, size_t dev_bytes, void* cuda_stream);
/* Point the handle at a device image that *_upload wrote earlier and that was then copied, byte
 * for byte, to `dev_buf` (same device).  No copy is made.  That copy must be COMPLETE (synchronised, or
 * made by an earlier operation of the stream the products will run on whose kernels have finished) before
 * the first product on it: the product kernels start reading the format ahead of stream order (see
 * hac_dot). */
int hac_attach (hac_format*  f, void* dev_buf, size_t dev_bytes);
int shac_attach(shac_format* f, void* dev_buf, size_t dev_bytes);

/* ---------------------------------------------------------------------------------------------
 * hac_dot / shac_dot - Algorithms 1, 2 (one input) and 3 (a batch), on the device:
 *       y[b*y_stride_b + j*y_stride_j] = sum_i W[i][j] * x[b*x_stride_b + i*x_stride_i]
 * for b in [0, batch), j in [0, m).  x, y: device fp32; strides in elements, so X may be stored
 * [batch][n] or [n][batch] and Y [batch][m] or [m][batch]; the batched kernels are fastest with
 * x_stride_b == 1 and y_stride_b == 1 (a HAC format built with sub-segments of several hundred symbols does
 * not fit the batched kernel's buffers and is then multiplied input by input).  x and y must not overlap.  Code words are decoded on the
 * fly; the uncompressed weights are never written to global memory.  Products and sums are fp32.
 *   workspace  device scratch of at least *_workspace_bytes(f, batch) bytes, 16-byte aligned (may be
 *              NULL when that is 0).  It holds partial sums of columns that span several segments
 *              and, for a batched product on the tensor cores (HAC always; sHAC when that is estimated
 *              to be faster than gathering rows of X), the inputs split into two TF32 parts and
 *              arranged in the tiles that kernel reads (for very large HAC matrices also the start bit
 *              of every sub-segment of every column, which is otherwise kept in the device image); its
 *              contents need not be initialised and are undefined afterwards.  Two dot calls that run
 *              concurrently must not share it.
 *   results    A batched product on the tensor cores rounds every weight and input to two TF32 parts
 *              (three partial products, error about 1e-7 of sum |w x|).  If a bounded wait inside
 *              that kernel ever ran out (it never has), the outputs of the affected block are NaN.
 *              x is expected to be finite.  A NaN or Inf in x[i] reaches every output whose column stores row i,
 *              as the definition says, and may also reach outputs whose column has a zero there: HAC multiplies
 *              its coded zeros (except where a run of them is skipped), the tensor-core tiles and the batched sHAC
 *              kernel pad with zero weights, and 0 * Inf is NaN.
 * Asynchronous on cuda_stream.  The kernels are launched with programmatic stream serialization:
 * they may begin fetching the uploaded format while the kernel before them in the stream is still
 * finishing, but read x and the workspace and write y only once that kernel has completed, so the
 * usual stream ordering holds for everything the caller can observe.  Errors: HAC_ERR_NOT_UPLOADED, HAC_ERR_INVALID_ARG (batch < 1, null
 * pointers, misaligned workspace), HAC_ERR_BUFFER_TOO_SMALL, HAC_ERR_CUDA (launch failure).
 * ------------------------------------------------------------------------------------------- */
int hac_workspace_bytes (const hac_format*  f, int64_t batch, size_t* out);
int shac_workspace_bytes(const shac_format* f, int64_t batch, size_t* out);
int hac_dot (const hac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b,
             float* y, int64_t y_stride_j, int64_t y_stride_b,
             void* workspace, size_t workspace_bytes, void* cuda_stream);
int shac_dot(const shac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b,
             float* y, int64_t y_stride_j, int64_t y_stride_b,
             void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Layer evaluation on the compressed format (Sect. V: the networks are evaluated with their fully
 * connected layers kept in HAC / sHAC): the product of hac_dot / shac_dot with the layer's bias and
 * activation applied to every output before it is stored, in the same kernels,
 *       y[b][j] = act( sum_i W[i][j] x[b][i] + bias[j] ),   act = identity or max(., 0).
 *   epilogue   NULL = plain product.  bias: device, m floats, or NULL; relu: 0 / 1; reserved: 0.
 * Everything else as hac_dot.
 * hac_chain evaluates a stack of such layers as one chained submission on cuda_stream (layer l + 1 may
 * begin fetching its format while layer l finishes, see hac_dot): layers[l] names a HAC or an sHAC handle
 * (exactly one non-NULL) and its epilogue; layer l's m must equal layer l + 1's n.  x is [n_0][batch] and y
 * [m_last][batch] with the inputs of a batch contiguous (plain vectors for batch 1); act0 / act1 are two
 * device buffers of act_floats floats each that take the intermediate activations in turn (act0 may be
 * NULL for one layer, act1 for at most two); the workspace must satisfy every layer's *_workspace_bytes.
 * After the call *_last_launch_count of the LAST layer's handle gives the launches of the whole chain.
 * ------------------------------------------------------------------------------------------- */
typedef struct hac_epilogue {
    const float* bias;     /* device, one per output (column of W), or NULL                       */
    uint32_t relu;         /* 1: negative results become 0                                        */
    uint32_t reserved;     /* must be 0                                                           */
} hac_epilogue;
typedef struct hac_layer {
    const hac_format*  hac;    /* the layer's weights as HAC ...                                   */
    const shac_format* shac;   /* ... or as sHAC (exactly one of the two)                          */
    hac_epilogue epilogue;
} hac_layer;
int hac_dot_layer (const hac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b,
                   float* y, int64_t y_stride_j, int64_t y_stride_b, const hac_epilogue* epilogue,
                   void* workspace, size_t workspace_bytes, void* cuda_stream);
int shac_dot_layer(const shac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b,
                   float* y, int64_t y_stride_j, int64_t y_stride_b, const hac_epilogue* epilogue,
                   void* workspace, size_t workspace_bytes, void* cuda_stream);
int hac_chain(const hac_layer* layers, int n_layers, const float* x, int64_t batch, float* y,
              float* act0, float* act1, size_t act_floats, void* workspace, size_t workspace_bytes,
              void* cuda_stream);

/* The same product for HOST inputs and outputs (Algorithm 3's calling convention: X is batch x n,
 * one input per row, Y is batch x m, both contiguous host fp32, ideally pinned).  The caller gives a
 * device staging buffer `dev_scratch` of at least *_dot_host_scratch_bytes(f, batch) bytes; the call
 * copies X to the device, runs the product, copies Y back and waits for cuda_stream.
 * *_dot_host_async enqueues the same three steps and returns without waiting: Y_host is valid, and
 * X_host, Y_host and dev_scratch may be reused, once the caller has synchronised cuda_stream.  Two
 * streams with a staging buffer each let the copies of one product overlap the kernels of another. */
int hac_dot_host_scratch_bytes (const hac_format*  f, int64_t batch, size_t* out);
int shac_dot_host_scratch_bytes(const shac_format* f, int64_t batch, size_t* out);
int hac_dot_host (const hac_format*  f, const float* X_host, int64_t batch, float* Y_host,
                  void* dev_scratch, size_t dev_scratch_bytes, void* cuda_stream);
int shac_dot_host(const shac_format* f, const float* X_host, int64_t batch, float* Y_host,
                  void* dev_scratch, size_t dev_scratch_bytes, void* cuda_stream);
int hac_dot_host_async (const hac_format*  f, const float* X_host, int64_t batch, float* Y_host,
                        void* dev_scratch, size_t dev_scratch_bytes, void* cuda_stream);
int shac_dot_host_async(const shac_format* f, const float* X_host, int64_t batch, float* Y_host,
                        void* dev_scratch, size_t dev_scratch_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * hac_dot_noalloc - the HAC product of hac_dot for callers that cannot hand over a workspace.
 * (The paper has no counterpart: this is a packaging variant of hac_dot, not a different method.)
 *
 * hac_dot needs a device workspace whenever a column of W spans several segments, and the caller has
 * to get that memory from somewhere.  Some hosts cannot: an inference server that carves up all
 * device memory at start-up and forbids later cudaMalloc calls (they serialise the device and can
 * fail under fragmentation), or a plugin that runs inside another program's memory plan and owns no
 * allocator at all.  For them this call keeps the partial sums in a buffer that is part of the
 * library image itself: a file-scope device array of HAC_NOALLOC_SCRATCH_BYTES bytes, present on
 * every GPU that loads the library until the process exits.  The call makes no cudaMalloc / cudaFree
 * and uses no allocating library routine; x and y are still the caller's.
 *
 * Arguments and result as hac_dot, without the workspace pair.
 *   - A product whose workspace would exceed HAC_NOALLOC_SCRATCH_BYTES (see hac_workspace_bytes)
 *     is refused with HAC_ERR_BUFFER_TOO_SMALL and nothing is launched; hac_last_cuda_error() then
 *     names the two sizes.  Use hac_dot with your own workspace for those.
 *   - The first call on each device looks up the device address of the buffer (one
 *     cudaGetSymbolAddress with that device current).  Make that first call outside any stream
 *     capture.
 *   - All calls on a device share the one buffer, and it keeps whatever the previous call left there.
 *     Nothing in it has to start at zero: every slot the finishing kernel reads is written by the
 *     product kernel of the same call first.  Two calls that may overlap on the GPU (different
 *     streams, or different handles on different threads) race on it and give wrong sums; run them on
 *     one stream, or order them with events.
 * ------------------------------------------------------------------------------------------- */
#define HAC_NOALLOC_SCRATCH_BYTES (4u << 20)
int hac_dot_noalloc(const hac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b,
                    float* y, int64_t y_stride_j, int64_t y_stride_b, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * The two formats HAC and sHAC are compared with: the index map (Sect. III-C.1) and plain CSC
 * (Sect. IV-A), each with its encoder on the host and its product on the device.  They take no handle:
 * the caller owns every array.
 *
 * hac_index_map_encode - the k distinct values of Wq (row-major, leading dimension ldw; zero is a
 *   value like any other; -0.0 counts as 0) ascending into codebook (room for 2^index_bits floats),
 *   their number into *k, and for every weight the position of its value into index_colmajor
 *   (index_colmajor[j*n + i] points at Wq[i][j]; uint8_t for index_bits == 8, uint16_t for 16; n*m
 *   entries).  All host memory.  Occupancy as the paper counts it: index_bits / 32 + k / (n m).
 *   Errors: HAC_ERR_INVALID_ARG, HAC_ERR_NONFINITE_INPUT, HAC_ERR_K_TOO_LARGE (more than 2^index_bits
 *   values), HAC_ERR_ALLOC.
 * hac_index_map_dot - y = x^T W with W[i][j] = codebook[index[j*n + i]], all pointers device memory,
 *   x and y with the strides of hac_dot, fp32 products and sums, asynchronous on cuda_stream.  A
 *   pointer at or beyond k reads the last codebook entry (two-byte pointers) or 0 (one-byte pointers).
 *   128-bit loads of the pointers are used when n is a multiple of 16 (one-byte pointers) or 8 (two-byte)
 *   and index_dev is 16-byte aligned; otherwise element loads.  Needs no workspace.
 *
 * shac_csc_encode - CSC of Wq: the nonzero weights column by column, rows ascending, into nz, their rows
 *   into ri, and the m+1 column boundaries into cb; their number into *q.  With nz, ri and cb all NULL
 *   only *q is written (size query); otherwise capacity is the room in nz and ri (entries).  Occupancy
 *   as the paper counts it: (2 q + m + 1) / (n m).  Errors: HAC_ERR_INVALID_ARG, HAC_ERR_NONFINITE_INPUT,
 *   HAC_ERR_BUFFER_TOO_SMALL, HAC_ERR_OFFSET_OVERFLOW (2^32 entries or more).
 * shac_csc_dot - y[j] = sum over p in [cb[j], cb[j+1]) of nz[p] * x[ri[p]], device pointers, strides as
 *   hac_dot, asynchronous on cuda_stream; a row at or beyond n contributes nothing.  nz_dev and ri_dev may
 *   be NULL when nothing is stored.
 * Both products: HAC_ERR_INVALID_ARG (null pointers, sizes below 1), HAC_ERR_CUDA (launch failure).
 * ------------------------------------------------------------------------------------------- */
int hac_index_map_encode(const float* Wq, int64_t n, int64_t m, int64_t ldw, int index_bits, void* index_colmajor,
                         float* codebook, int* k);
int hac_index_map_dot(const void* index_dev, int index_bits, const float* codebook_dev, int k, int64_t n, int64_t m,
                      const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b, float* y,
                      int64_t y_stride_j, int64_t y_stride_b, void* cuda_stream);
int shac_csc_encode(const float* Wq, int64_t n, int64_t m, int64_t ldw, float* nz, uint32_t* ri, uint32_t* cb,
                    int64_t capacity, int64_t* q);
int shac_csc_dot(const float* nz_dev, const uint32_t* ri_dev, const uint32_t* cb_dev, int64_t n, int64_t m, const float* x,
                 int64_t batch, int64_t x_stride_i, int64_t x_stride_b, float* y, int64_t y_stride_j, int64_t y_stride_b,
                 void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * TEST ONLY: decode on the device into a caller's device buffer, to show that the kernels' decoder
 * reproduces the quantized weights bit for bit (the formats are lossless, Sect. IV-B).  The product
 * path never does this.  hac: W_colmajor[j*n + i] = Wq[i][j] (n*m floats).  shac: nz[p] for the nnz
 * stored entries in CSC order.  Asynchronous on cuda_stream.
 * ------------------------------------------------------------------------------------------- */
int hac_debug_decode (const hac_format*  f, float* W_colmajor_dev, void* cuda_stream);
int shac_debug_decode(const shac_format* f, float* nz_dev, void* cuda_stream);

/* TEST ONLY, host: what the kernels' first-level decoding table holds for a 32-bit window of the stream
 * (most significant bit = next bit to decode): *length = 0 if the entry leaves the code word to the slower
 * levels, else the code word's length and *value the shared value it stands for (Sect. IV-B: the inverse
 * dictionary H^-1).  *kind = 0 for the table indexed by the leading bits, 1 for the one indexed by the
 * magnitude of the inverted window; *never_unresolved = 1 if the kernels rely on every window being resolved. */
int hac_debug_table_lookup (const hac_format*  f, uint32_t window, float* value, uint32_t* length, int* kind,
                            int* never_unresolved);
int shac_debug_table_lookup(const shac_format* f, uint32_t window, float* value, uint32_t* length, int* kind,
                            int* never_unresolved);

/* Number of kernels the last dot / debug call on this handle launched (for launch accounting). */
int hac_last_launch_count (const hac_format*  f);
int shac_last_launch_count(const shac_format* f);

void hac_free (hac_format*  f);
void shac_free(shac_format* f);

const char* hac_status_string(int status);
/* Text of the last CUDA error seen by this library on the calling thread ("" if none). */
const char* hac_last_cuda_error(void);

/* Number of thread blocks of the batched tensor-core kernel, on the current device since the library was loaded, in which
 * a bounded wait ran out (the affected outputs were set to NaN, see hac_dot).  0 is the only value ever observed; a caller that
 * finds NaN in y can tell a lost wait from NaN inputs with it.  Synchronous: a cudaMemcpyFromSymbol, which waits for the
 * device work submitted before it on blocking streams.  Errors: HAC_ERR_INVALID_ARG, HAC_ERR_CUDA. */
int hac_lost_waits(unsigned int* count);

/* Diagnostic switches.  Environment variables, read once when the first product is launched (changing
 * them later has no effect); they select between code paths that all give the same results:
 *   HAC_B200_PDL=0          launch without programmatic stream serialization
 *   HAC_B200_ROWS=0         single-input HAC always through the kernel that keeps x in shared memory
 *   HAC_B200_ROWS_WARPS=n   warps per block of the rows-in-registers kernel (default: chosen per format)
 *   HAC_B200_ROWS_CHAINS=c  decode chains per lane of that kernel, 2 or 3 (default 2)
 *   HAC_B200_PREFETCH=1     that kernel requests its block's share of the stream into L2 at its start (default off)
 *   HAC_B200_VEC_GROUP=0    the kernel that keeps x in shared memory decodes one code word per table lookup
 *   HAC_B200_VEC_WARPS=n    warps per block of the kernels that keep x in shared memory (default: as many as fit)
 *   HAC_B200_ITEMS=0        single-input sHAC always through the older kernel
 *   HAC_B200_SHAC_TC=0|2    batched sHAC never / always on the tensor cores (default 1: by estimated cost)
 *   HAC_B200_GEMM_CLUSTER=0 batched HAC adds its row splits in a finishing kernel instead of a thread-block cluster
 *   HAC_B200_SHAC_ROWS=0     batched sHAC never through the kernel that stages rows of X in shared memory; 2: whenever it can
 *   HAC_B200_SHAC_ROWS_GROUP=n  row tasks per staged group of that kernel (0 = chosen by the library)
 *   HAC_B200_ZERO_RUNS=0    never use the zero-run table of mostly-zero HAC streams
 *   HAC_B200_XT=0           never use the magnitude-indexed first-level table */

#ifdef __cplusplus
}
#endif
#endif  /* HAC_H_ */
