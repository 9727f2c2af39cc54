/*
 * dnns.h - C ABI of the sparse-to-pruned conversion path of DNNShifter on one GPU.
 *
 * The path turns a dense CNN into a portfolio of smaller model variants:
 *
 *   dnns_magnitude_threshold  rank the prunable weights by magnitude and find, for every
 *                             requested prune count k, the k-th smallest magnitude
 *                             (Phase 1's "unstructured ranking", Section III-C; a compression
 *                             ratio C leaves C-1 of every C weights zero, Section IV-B-1);
 *   dnns_apply_mask           set the k weights of least magnitude to zero - the sparse model,
 *                             which is not yet smaller (Section III-C);
 *   dnns_zero_structures      Module 2, Sparsity Analyser: all-zero 2-D kernels, then the
 *                             channels all of whose kernels are zero (Section III-D, Figure 2);
 *   dnns_propagate_keep       Module 3, Prune Planner (Algorithm 1): which channels every layer
 *                             drops, planned for all layers at once;
 *   dnns_compact              Module 4, Model Pruner (Algorithm 2): rebuild every layer without
 *                             its prunable in/out channels, biases and BatchNorm entries, all
 *                             layers in one batch.
 *
 * General rules
 *   - Every function returns a dnns_status; nothing throws, aborts or traps.  Argument and
 *     graph errors are found on the host before anything is launched.
 *   - "device" pointers are CUDA device memory of the current device, owned by the caller.
 *     The library allocates no device memory: tables and scratch live in the caller's
 *     workspace (dnns_workspace_bytes).  Host pointers are only read during the call.
 *   - Every compute call enqueues its kernels on `stream` (a cudaStream_t passed as void*,
 *     NULL = the default stream) and returns without synchronising.  Only
 *     dnns_last_device_status and dnns_plan_destroy synchronise.
 *   - Calls on one plan must be issued in stream order on one stream at a time: the plan's
 *     workspace is shared state.
 *
 * Layouts
 *   - Weights are OIHW, contiguous, row-major: filter o is I*KH*KW consecutive elements, the
 *     2-D kernel (o,i) is KH*KW consecutive elements.  A fully-connected layer is [O][I] with
 *     KH = KW = 1 and I = C_in*in_spatial; the columns of input channel c are
 *     c*in_spatial .. (c+1)*in_spatial-1.  Tensor data pointers must be 16-byte aligned.
 *   - A magnitude is compared as the stored word with its sign bit cleared (31-bit keys for
 *     fp32, 15-bit keys for bf16), as an unsigned integer: -0 equals +0, denormals order
 *     numerically, infinities lie above all finite values, NaNs above those.  A weight is
 *     "zero" when that key is 0.
 *   - Bit sets are uint32 words, bit b in word b/32 at position b%32.  Per-tensor and
 *     per-group bit sets and index lists are packed one after another into ONE device array
 *     each, at the word/element offsets dnns_plan_layout reports (each set starts on a word).
 *   - A "masked arena" holds a copy of every weight tensor of the model at the byte offsets
 *     dnns_plan_layout reports (256-byte aligned, descriptor order).
 */
#ifndef DNNS_H
#define DNNS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DNNS_OK = 0,
    DNNS_ERR_INVALID_ARG = 1, /* null pointer, non-positive extent, misaligned data, k above its segment */
    DNNS_ERR_BAD_GRAPH = 2,   /* tensor / BN / group extents that do not agree                             */
    DNNS_ERR_WORKSPACE = 3,   /* workspace or destination arena too small                                   */
    DNNS_ERR_UNSUPPORTED = 4, /* mixed dtypes, unknown dtype, extents beyond the documented limits          */
    DNNS_ERR_CUDA = 5,        /* a CUDA runtime call failed                                                 */
    DNNS_ERR_TIMEOUT = 6,     /* a bounded device-side wait ran out (device status of the rebuild)          */
    DNNS_ERR_STATIC_LIMIT = 7 /* input larger than the built-in scratch of a *_static entry point allows    */
} dnns_status;

typedef enum { DNNS_F32 = 0, DNNS_BF16 = 1 } dnns_dtype;
typedef enum { DNNS_SCOPE_GLOBAL = 0, DNNS_SCOPE_PER_TENSOR = 1 } dnns_scope;

/* policy bits of dnns_propagate_keep */
enum { DNNS_RULE_PRODUCER = 1, DNNS_RULE_CONSUMER = 2, DNNS_SHIFT_STRICT = 4 };
/* group flags */
enum { DNNS_GROUP_FROZEN = 1 };

/* One weight tensor.  out_group / in_group name the channel groups of its two axes. */
typedef struct {
    void* data;         /* device, 16-byte aligned, O*I*KH*KW elements of `dtype`            */
    int32_t dtype;      /* dnns_dtype; all tensors of a model share one dtype                 */
    int32_t O, I, KH, KW;
    int32_t in_spatial; /* S: columns per input channel (1 for convs and after global pooling)*/
    int32_t prunable;   /* takes part in ranking and masking                                  */
    int32_t out_group;  /* group of the O axis; O == groups[out_group].C                      */
    int32_t in_group;   /* group of the I axis; I == groups[in_group].C * in_spatial          */
    float* bias;        /* device, fp32, length O; NULL when the layer has none               */
} dnns_tensor;

/* BatchNorm following conv `tensor`; its vectors follow that tensor's out-axis. */
typedef struct {
    float *gamma, *beta, *mean, *var; /* device, fp32, length C */
    int32_t C;
    int32_t tensor;
    float eps;
} dnns_bn;

/* A set of channels shared by the out-axes that write it (producers) and the in-axes that
 * read it (consumers): one layer boundary in a chain, a whole residual stream in a ResNet. */
typedef struct {
    int32_t C;
    uint32_t flags; /* DNNS_GROUP_FROZEN: never pruned (network input, class axis) */
} dnns_group;

typedef struct {
    int32_t n_tensors;
    const dnns_tensor* tensors;
    int32_t n_bn;
    const dnns_bn* bns;
    int32_t n_groups;
    const dnns_group* groups;
} dnns_model;

/* Result of the ranking for one (variant, segment). */
typedef struct {
    uint32_t tau_bits; /* magnitude key of the k-th smallest weight                  */
    uint32_t pad;
    uint64_t n_below;  /* weights whose key is below tau                             */
    uint64_t n_tie;    /* k - n_below: weights equal to tau that are masked (>= 1)   */
    uint64_t n_equal;  /* weights whose key equals tau                               */
} dnns_threshold;     /* k == 0 gives the all-zero record                           */

/* Sizes and offsets of the packed buffers, all host memory owned by the plan. */
typedef struct {
    int32_t n_tensors, n_bn, n_groups, n_segments, n_bias;
    int32_t elem_bytes;            /* 4 or 2                                                        */
    uint64_t n_prunable;           /* prunable weights in the model                                 */
    uint64_t masked_arena_bytes;   /* size of a masked arena                                        */
    uint64_t mask_words;           /* uint32 words of the packed mask bits (numel bits per tensor)  */
    uint64_t nz_map_words;         /* packed kernel maps (O*I bits per tensor)                      */
    uint64_t out_nz_words;         /* packed out flags (O bits per tensor)                          */
    uint64_t in_nz_words;          /* packed in flags (I bits per tensor)                           */
    uint64_t keep_words;           /* packed keep bits (C bits per group)                           */
    uint64_t keep_idx_len;         /* packed keep index lists (C entries per group)                 */
    uint64_t compact_arena_bytes;  /* worst-case size of a destination arena for dnns_compact       */
    int32_t n_compact_items;       /* n_tensors + 4*n_bn + n_bias                                   */
    const uint64_t* arena_offset;  /* [n_tensors] byte offset of tensor t in a masked arena         */
    const uint64_t* mask_offset;   /* [n_tensors] word offsets into the packed arrays ...           */
    const uint64_t* nz_map_offset; /* [n_tensors]                                                   */
    const uint64_t* out_nz_offset; /* [n_tensors]                                                   */
    const uint64_t* in_nz_offset;  /* [n_tensors]                                                   */
    const uint64_t* keep_offset;   /* [n_groups] word offset of the group's keep bits               */
    const uint64_t* keep_idx_offset; /* [n_groups] element offset of the group's index list         */
    const uint64_t* segment_size;  /* [n_segments] prunable weights per ranking segment             */
    const int32_t* segment_of_tensor; /* [n_tensors] segment index, -1 when not prunable            */
} dnns_layout;

typedef struct dnns_plan dnns_plan; /* opaque; host object */

/* Device bytes a plan needs for `max_variants` prune counts per segment.  0 on invalid input. */
size_t dnns_workspace_bytes(const dnns_model* model, dnns_scope scope, int32_t max_variants);

/*
 * Validate the model (host descriptors holding device pointers), build the tile, segment and
 * group tables and upload them into the workspace.  scope fixes the ranking segments
 * (Section III-C leaves global or per-layer ranking open: GLOBAL = one segment of all prunable
 * weights in descriptor order, PER_TENSOR = one segment per prunable tensor).
 * ws_dev must be 256-byte aligned and stay valid and untouched until the plan is destroyed.
 * Errors: INVALID_ARG, BAD_GRAPH (an out-axis whose O differs from its group's C, an in-axis
 * whose I differs from C*in_spatial, a BN whose C differs from its tensor's O, two BNs on one
 * tensor), UNSUPPORTED (mixed or unknown dtype, a tensor of 2^31 or more elements, a segment
 * of 2^32 or more weights, a group above 65536 channels, max_variants outside 1..64),
 * WORKSPACE, CUDA.
 */
dnns_status dnns_plan_create(const dnns_model* model, dnns_scope scope, int32_t max_variants, void* ws_dev,
                             size_t ws_bytes, void* stream, dnns_plan** plan_out);
/* Synchronises the device, then frees the host object.  The workspace stays the caller's. */
void dnns_plan_destroy(dnns_plan* plan);
dnns_status dnns_plan_layout(const dnns_plan* plan, dnns_layout* out);
/* Kernels this plan has launched so far (memsets and copies not counted). */
uint64_t dnns_plan_launch_count(const dnns_plan* plan);

/*
 * Per-kernel timing of a plan's calls, for reports (the paper's Module 5 profiles models; this profiles
 * the conversion itself).  dnns_plan_profile(plan, 1) synchronises the device, drops earlier records and,
 * from then on, brackets every kernel the plan's calls launch with a pair of CUDA events on the launching
 * stream (two event creations per launch: host work, so switch it off for timed runs and do not switch it
 * on while a stream is being captured); dnns_plan_profile(plan, 0) stops recording.
 * dnns_plan_profile_read synchronises the device and returns the summed device time and the number of
 * recorded launches of the kernels whose name starts with `kernel` ("k_sweep", "k_compact_gather",
 * "k_flags", "k_shift_zero", "k_propagate", "k_rebuild_layout", "k_hist1", "k_hist2", "k_ties", "k_select1", "k_select2",
 * "k_tie_scan", "k_tie_find", "k_tie_pick", "k_extrema_rows", "k_extrema_sweep", "k_extrema_flags").
 */
dnns_status dnns_plan_profile(dnns_plan* plan, int32_t enable);
dnns_status dnns_plan_profile_read(dnns_plan* plan, const char* kernel, double* total_ms, uint64_t* launches);

/*
 * For reports: whether the latest dnns_magnitude_threshold call read the weights once more to count, tile by tile,
 * the weights equal to tau (*swept = 1) or not (*swept = 0).  With 32-bit weights the second ranking sweep lists the
 * keys it counts together with their positions, and the place where a variant stops masking the weights equal to
 * tau is then found in that list; the extra sweep runs only when no list is kept (16-bit weights; plans with more
 * than 255 segments or more than 1024 (variant, segment) pairs), when a list cannot answer (it ran over, tau is
 * zero, or more than 1024 weights equal tau), or later, on demand, when a sweep that masks tile by tile
 * (dnns_apply_mask, dnns_mask_and_structures, dnns_mask_and_structures_multi) needs the per-tile tables.  Never when
 * no variant masks only part of the weights equal to tau.  Synchronises the device.
 * Errors: INVALID_ARG (null), CUDA.
 */
dnns_status dnns_plan_tie_sweep(dnns_plan* plan, int32_t* swept);

/*
 * Step 1 - exact k-th-magnitude threshold by radix select over the magnitude keys.
 * k (host): k[v*n_segments + s] = how many weights of segment s variant v masks, 0 <= k <= the
 * segment's size, 1 <= n_k <= max_variants.  thr_dev (device, n_k*n_segments records, same
 * indexing) receives the records.  One call serves the whole portfolio: the sweeps over the
 * weights are shared by all n_k counts.  The call also leaves, in the workspace, the place
 * (tensor, element) where each variant stops masking the weights equal to tau, which
 * dnns_compact_masked reads (the per-tile tables of those weights, which dnns_apply_mask needs to
 * mask exactly k weights tile by tile, are made by the call itself or, see dnns_plan_tie_sweep,
 * by the first such sweep after it), and the largest key of every filter and every input column of every
 * tensor, which dnns_zero_structures_portfolio reads (one more sweep over the weights, enqueued on a
 * stream of the plan's own that forks from `stream` at the start of the call and joins it again at
 * the end, so that it runs beside the ranking kernels; a call inside a stream capture records that
 * fork and join as well).  All of these belong to this call's thr_dev and to the weights as they
 * were during the call.
 * Errors: INVALID_ARG (null, n_k out of range, a k above its segment), CUDA.
 */
dnns_status dnns_magnitude_threshold(dnns_plan* plan, const uint64_t* k, int32_t n_k, dnns_threshold* thr_dev,
                                     void* stream);

/*
 * Step 2 - mask variant `variant` of the latest dnns_magnitude_threshold call on this plan
 * (thr_dev is that call's output array).  A weight is masked when its key is below tau, or
 * equals tau and fewer than n_tie equal weights precede it in the segment (tensors in
 * descriptor order, row-major inside): exactly k weights per segment.  Masked weights become
 * +0, the others are copied bit for bit; tensors that are not prunable are copied.
 * masked_arena (device): destination in arena layout, or NULL to mask the model's tensors in
 * place (only meaningful for the weights the thresholds were computed on).  variant must be one of
 * the latest threshold call's (INVALID_ARG otherwise; the same holds for every call that takes one).
 * mask_bits (device, nullable): packed mask bits, 1 = kept; padding bits are written as 0.
 */
dnns_status dnns_apply_mask(dnns_plan* plan, const dnns_threshold* thr_dev, int32_t variant, void* masked_arena,
                            uint32_t* mask_bits, void* stream);

/*
 * Step 3 - zero structures of a sparse model.  masked_arena (device): the weights to analyse in
 * arena layout, or NULL for the model's own tensors (a sparse model that arrived from training).
 * Per tensor: nz_map (nullable) bit o*I+i = kernel (o,i) has a non-zero element; out_nz bit o =
 * filter o has one; in_nz bit i = some filter reads input column i.  All three are packed device
 * arrays (see dnns_layout) and are fully overwritten.
 */
dnns_status dnns_zero_structures(dnns_plan* plan, const void* masked_arena, uint32_t* nz_map, uint32_t* out_nz,
                                 uint32_t* in_nz, void* stream);

/*
 * Steps 2 and 3 in one sweep over the weights: the same outputs, bit for bit, as dnns_apply_mask
 * followed by dnns_zero_structures on its result, but the masked weights are analysed while they
 * are still in registers, which saves one full read of the model per variant (Module 2 only
 * needs the sparse weights, Section III-D).  Arguments as in the two calls; masked_arena NULL
 * masks in place.
 */
dnns_status dnns_mask_and_structures(dnns_plan* plan, const dnns_threshold* thr_dev, int32_t variant,
                                     void* masked_arena, uint32_t* mask_bits, uint32_t* nz_map, uint32_t* out_nz,
                                     uint32_t* in_nz, void* stream);

/*
 * Steps 2 and 3 for up to DNNS_MULTI_MAX variants of the latest threshold call in ONE sweep over the
 * dense weights: variants first_variant .. first_variant + n_variants - 1, each with outputs of its own,
 * bit for bit what dnns_mask_and_structures gives for that variant.  The portfolio's variants all start
 * from the same dense model (Section III-C: every iteration's sparse model joins the portfolio), so the
 * model is read once per group of variants instead of once per variant.
 * masked_arenas, out_nz, in_nz: host arrays of n_variants device pointers, all distinct; mask_bits, nz_map:
 * host arrays of n_variants device pointers, or NULL (entries of mask_bits may be NULL too).  In-place
 * masking is not offered here.
 * When every entry of masked_arenas is NULL the masked weights are not written at all: the call then leaves
 * only the mask bits (required in that case, one array per variant) and the zero structures, and
 * dnns_compact_masked rebuilds a variant straight from the dense model - the sparse model of Section III-C,
 * which is as large as the dense one, is never stored.  Errors: INVALID_ARG, CUDA.
 */
#define DNNS_MULTI_MAX 4
dnns_status dnns_mask_and_structures_multi(dnns_plan* plan, const dnns_threshold* thr_dev, int32_t first_variant,
                                           int32_t n_variants, void* const* masked_arenas, uint32_t* const* mask_bits,
                                           uint32_t* const* nz_map, uint32_t* const* out_nz, uint32_t* const* in_nz,
                                           void* stream);

/*
 * Step 3 for up to DNNS_PORTFOLIO_MAX variants of the latest threshold call without a sweep of its own and
 * without forming any sparse model.  Step 2 keeps a weight of variant v when its key lies above tau_v
 * (or equals it and is not among the first n_tie such weights), so a filter or an input column still holds a
 * non-zero weight for v exactly when the largest key in it does: the threshold call recorded the largest key of
 * every filter and every input column (in the workspace), and each variant's flags follow from comparing those with
 * its threshold; where a maximum equals tau in the tensor in which the variant's equal weights split, that one
 * filter or column is read again.  out_nz, in_nz: host arrays of n_variants device pointers, all distinct, each
 * as in dnns_zero_structures and bit for bit what dnns_apply_mask + dnns_zero_structures give for variant
 * first_variant + i.  Kernel maps and mask bits are not produced here.  Follow with dnns_propagate_keep_multi
 * and, per variant, dnns_compact_masked: the sparse model of Section III-C is never stored.
 * Errors: INVALID_ARG (null, count or range outside the latest threshold call, repeated buffers), CUDA.
 */
#define DNNS_PORTFOLIO_MAX 16
dnns_status dnns_zero_structures_portfolio(dnns_plan* plan, const dnns_threshold* thr_dev, int32_t first_variant,
                                           int32_t n_variants, uint32_t* const* out_nz, uint32_t* const* in_nz,
                                           void* stream);

/*
 * Step 4 - keep sets per channel group (Algorithm 1 generalised from a chain to groups).
 * Channel j of a group is removed when
 *   (policy & RULE_PRODUCER) and every producer's filter j is all zero [the paper's rule], and,
 *       under SHIFT_STRICT, the constant each of those zero filters still emits through its
 *       BatchNorm / bias is structurally zero (beta == 0 and (gamma == 0 or mean == bias); no BN:
 *       bias == 0); or
 *   (policy & RULE_CONSUMER) and no consumer has a non-zero weight in the columns of channel j.
 * Frozen groups keep everything.  If fewer than min(min_keep, C) channels stay, removed channels
 * are taken back in ascending order.  Single pass, nothing is re-evaluated after removal.
 * Outputs (device, packed per group): keep_bits, keep_idx (kept channels ascending; entries past
 * keep_count are left untouched), keep_count [n_groups].  The call also prepares, in the workspace, the
 * destination layout of step 5 for these counts (one more small kernel); dnns_compact finds it by the address
 * of keep_count, so leave that array as this call wrote it until the rebuild has been enqueued.
 * stats (device, nullable, 4 words):
 * [0] removed (producer, channel) pairs whose non-zero constant is dropped while some consumer
 * still reads the channel, [1] channels removed, [2] channels taken back by min_keep, [3] 0.
 */
dnns_status dnns_propagate_keep(dnns_plan* plan, const uint32_t* out_nz, const uint32_t* in_nz, uint32_t policy,
                                int32_t min_keep, uint32_t* keep_bits, int32_t* keep_idx, int32_t* keep_count,
                                uint64_t* stats, void* stream);

/*
 * Step 4 for n_variants (1..DNNS_PORTFOLIO_MAX) variants - those of a dnns_mask_and_structures_multi or
 * dnns_zero_structures_portfolio call - in one launch:
 * Algorithm 1 plans all layers of a model at once; the variants of a portfolio are independent models, so they
 * are planned at once too.  out_nz, in_nz, keep_bits, keep_idx, keep_count: host arrays of n_variants device
 * pointers (the outputs all distinct), each as in dnns_propagate_keep; stats (device, nullable): 4 words per
 * variant, contiguous.  Outputs per variant are bit for bit those of dnns_propagate_keep.
 */
dnns_status dnns_propagate_keep_multi(dnns_plan* plan, int32_t n_variants, const uint32_t* const* out_nz,
                                      const uint32_t* const* in_nz, uint32_t policy, int32_t min_keep,
                                      uint32_t* const* keep_bits, int32_t* const* keep_idx, int32_t* const* keep_count,
                                      uint64_t* stats, void* stream);

/*
 * Step 4 applied to a fixed point.  Algorithm 1 looks at the zero channels once; once channels are
 * gone, a filter whose only non-zero 2-D kernels sit in removed input channels is a zero channel
 * too, and an input column that only removed filters read is unread.  Pass p judges every channel by
 * the rule of dnns_propagate_keep on the kernel maps restricted to what pass p-1 kept (all channels
 * against the same previous sets; removal only grows); passes end when nothing changes or after
 * max_passes (1..64; pass 1 alone is dnns_propagate_keep).  min_keep is applied once, at the end.
 * nz_map (device): the packed kernel maps written by dnns_zero_structures / dnns_mask_and_structures.
 * Outputs as in dnns_propagate_keep; stats[0] is judged in the last pass, stats[3] = passes that
 * removed something.  The launches of all max_passes passes are enqueued; those after the last
 * change return at once.
 */
dnns_status dnns_propagate_keep_cascade(dnns_plan* plan, const uint32_t* nz_map, uint32_t policy, int32_t min_keep,
                                        int32_t max_passes, uint32_t* keep_bits, int32_t* keep_idx,
                                        int32_t* keep_count, uint64_t* stats, void* stream);

/*
 * Step 5 - rebuild every tensor with its kept channels only (Algorithm 2):
 *   W'[a][c][s][y][x] = W[keep_out[a]][keep_in[c]][s][y][x],  v'[a] = v[keep_out[a]] for every
 * BatchNorm vector and bias.  masked_arena as in step 3.  The destination arena receives, at
 * 256-byte aligned offsets computed on the device from keep_count, first the n_tensors weight
 * tensors in descriptor order, then gamma, beta, mean, var of every BN in order, then the biases
 * of the tensors that have one.  dst_offsets_dev [n_compact_items] receives those byte offsets,
 * dst_shapes_dev [n_tensors][2] the new (O', I').  dst_bytes >= layout.compact_arena_bytes always
 * suffices; if the arena is too small for this variant nothing is copied and the device status
 * becomes DNNS_ERR_WORKSPACE.
 * keep_idx / keep_count are normally the outputs of a dnns_propagate_keep* call on this plan, which has
 * already laid the variant out; for any other array of counts the layout kernel is enqueued here first.
 * Weight tensors whose filters are multiples of 16 bytes long are moved through shared memory with bulk
 * copies that complete on barriers; every wait on such a barrier is bounded (half a second), and a wait that
 * runs out ends the kernel and leaves DNNS_ERR_TIMEOUT in the device status instead of hanging.
 */
dnns_status dnns_compact(dnns_plan* plan, const void* masked_arena, const int32_t* keep_idx,
                         const int32_t* keep_count, void* dst_arena, size_t dst_bytes, uint64_t* dst_offsets_dev,
                         int32_t* dst_shapes_dev, void* stream);

/*
 * Step 5 reading the DENSE model (the tensors of the plan's model) and applying step 2 on the way: a weight
 * is copied when its key lies above tau of its ranking segment, or equals tau and is not among the first n_tie
 * such weights of the segment, else +0 is written.  Bit for bit the result of dnns_apply_mask followed by
 * dnns_compact, without the sparse model ever being stored.  thr_dev / variant as in dnns_apply_mask: the
 * thresholds of the latest dnns_magnitude_threshold call on this plan, which also left in the workspace, for
 * every variant that masks only part of the weights equal to tau, the place where that part ends.  The
 * remaining arguments as in dnns_compact.
 */
dnns_status dnns_compact_masked(dnns_plan* plan, const dnns_threshold* thr_dev, int32_t variant,
                                const int32_t* keep_idx, const int32_t* keep_count, void* dst_arena, size_t dst_bytes,
                                uint64_t* dst_offsets_dev, int32_t* dst_shapes_dev, void* stream);

/*
 * dnns_compact_masked for n_variants (1..DNNS_PORTFOLIO_MAX) variants first_variant .. first_variant + n_variants - 1
 * in ONE launch: the variants of a portfolio are rebuilt from the same dense model and are independent of one
 * another, so their gathers share one grid, and a block that has finished its share of one variant goes on with
 * the next.  keep_idx, keep_count, dst_arenas, dst_offsets_dev, dst_shapes_dev: host arrays of n_variants device
 * pointers, entry i for variant first_variant + i, each as in dnns_compact_masked; the destinations (and the
 * arrays of counts) all distinct, every arena of dst_bytes.  Bit for bit n_variants calls of dnns_compact_masked.
 */
dnns_status dnns_compact_masked_multi(dnns_plan* plan, const dnns_threshold* thr_dev, int32_t first_variant,
                                      int32_t n_variants, const int32_t* const* keep_idx,
                                      const int32_t* const* keep_count, void* const* dst_arenas, size_t dst_bytes,
                                      uint64_t* const* dst_offsets_dev, int32_t* const* dst_shapes_dev, void* stream);

/*
 * Module 1, Model Pre-Processor (Section III-D): fold every BatchNorm into the convolution it
 * follows, on a rebuilt variant as dnns_compact left it (same dst_arena, dst_offsets_dev,
 * dst_shapes_dev).  In place, fp32 arithmetic (bf16 weights are widened, scaled, rounded to nearest
 * even):  s_o = gamma_o / sqrt(var_o + eps);  W[o] <- W[o] * s_o;  the arena slot of gamma receives
 * s, the slot of beta receives the folded bias beta_o + (bias_o - mean_o) * s_o (bias_o = 0 when the
 * layer has none).  mean and var are left as they are; tensors without BatchNorm are untouched.
 * Floating point: results agree with an fp64 evaluation to a few fp32 units in the last place.
 */
dnns_status dnns_fold_batchnorm(dnns_plan* plan, void* dst_arena, const uint64_t* dst_offsets_dev,
                                const int32_t* dst_shapes_dev, void* stream);

/*
 * Phase 3, Module 7 (Model Deflater) and the inflation of Module 8 (Section III-E): a rebuilt variant
 * that is not in use is packed with the lossless DEFLATE format (RFC 1951) - the zeroed weights that
 * survive the rebuild repeat - and unpacked when it is switched in.  Both calls work on plain byte
 * buffers (a destination arena of dnns_compact, or anything else) and need no plan.
 *
 * dnns_deflate writes a raw RFC 1951 stream that any inflater can read.  The encoder's choices:
 * the input is cut into chunks of DNNS_DEFLATE_CHUNK bytes, each one block (fixed Huffman codes, or
 * stored when that is shorter) followed - except after the last - by an empty stored block, so every
 * chunk starts on a byte boundary; inside a chunk, sub-blocks of DNNS_DEFLATE_SUB bytes are coded on
 * their own: every run of equal bytes is a literal followed by matches at distance 1 (258 at a time,
 * then one match of the 3..257 repeats left, else literals).  An empty input is one empty final block.
 *   src_dev (device, 16-byte aligned, n_bytes), stream_dev (device, 16-byte aligned, capacity at
 *   least dnns_deflate_bound(n_bytes) rounded up to 4), chunk_offset_dev (device,
 *   dnns_deflate_chunks(n_bytes) + 1 entries: byte offset of every chunk, the last entry is the
 *   stream's size), sub_bits_dev (device, 32 entries per chunk: bit offset, from the chunk's first
 *   byte, of the first token of every sub-block; for a stored chunk, of its first byte), ws_dev
 *   (device, 16-byte aligned scratch of dnns_deflate_workspace_bytes(n_bytes), contents undefined
 *   afterwards).  Enqueues three kernels on `stream`; nothing is read back.
 * dnns_inflate restores the n_bytes from a stream, its two index arrays and its size, all as
 * dnns_deflate left them (stream_dev readable up to stream_bytes rounded up to 4, dst_dev 16-byte
 * aligned).  It decodes the streams dnns_deflate writes, not arbitrary DEFLATE: a block type, symbol
 * or distance the encoder never emits sets *status_dev (device word, cleared by the caller) to
 * DNNS_ERR_UNSUPPORTED and leaves that sub-block incomplete; nothing traps.
 * Errors of both: INVALID_ARG (null or misaligned pointer), WORKSPACE (capacity or scratch too
 * small), UNSUPPORTED (more than 2^40 bytes), CUDA.
 */
#define DNNS_DEFLATE_CHUNK 16384
#define DNNS_DEFLATE_SUB 512
size_t dnns_deflate_chunks(size_t n_bytes);          /* max(1, ceil(n_bytes / DNNS_DEFLATE_CHUNK))   */
size_t dnns_deflate_bound(size_t n_bytes);           /* largest possible stream: n_bytes + 5 * chunks */
size_t dnns_deflate_workspace_bytes(size_t n_bytes); /* device scratch of dnns_deflate                */
dnns_status dnns_deflate(const void* src_dev, size_t n_bytes, void* stream_dev, size_t stream_capacity,
                         uint64_t* chunk_offset_dev, uint32_t* sub_bits_dev, void* ws_dev, size_t ws_bytes, void* stream);
dnns_status dnns_inflate(const void* stream_dev, size_t stream_bytes, const uint64_t* chunk_offset_dev,
                         const uint32_t* sub_bits_dev, size_t n_bytes, void* dst_dev, uint32_t* status_dev, void* stream);

/* Synchronises `stream`, then returns (and clears) the status recorded by the plan's kernels. */
dnns_status dnns_last_device_status(dnns_plan* plan, void* stream);

const char* dnns_status_string(dnns_status s);

/*
 * The threshold of step 1 for ONE tensor, for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a packaging variant of dnns_magnitude_threshold.)
 *
 * Meant for code that runs where cudaMalloc is off limits: a plug-in inside another framework's
 * memory-planned step, a callback invoked while that framework's allocator is locked, a process
 * whose device memory was fully handed out at start-up.  Such callers own the weights and the
 * result record but cannot supply the workspace a plan needs, so the histograms and tables live
 * in a fixed array inside the library (about 0.6 MB, held by every GPU that loads the library
 * until the process exits).  Apart from the first call on a device (below), a call makes no allocation of any
 * kind, on device or host: it enqueues one memset, one one-thread kernel that stores the call's descriptors
 * (they travel as kernel arguments, so a captured call replays with the arguments it was captured with) and the
 * kernels of the threshold step.
 *
 * weights_dev: device, 16-byte aligned, numel elements of dtype (DNNS_F32 / DNNS_BF16), treated as
 * one ranking segment in index order.  k: how many weights to mask, 0 <= k <= numel.  thr_dev:
 * device, one record, same meaning as in dnns_magnitude_threshold.
 * Limits and errors: numel > DNNS_STATIC_MAX_NUMEL returns DNNS_ERR_STATIC_LIMIT and launches
 * nothing; INVALID_ARG (null or misaligned pointer, numel == 0, k > numel), UNSUPPORTED (dtype,
 * device ordinal above 63), CUDA.
 * The first call on each device resolves the array's device address; it is also the moment at which the CUDA
 * runtime loads this library's device code and places the array, so make that call at start-up, before the
 * allocator is locked (k = 0 on any small buffer will do), and outside any stream capture: a first call on a
 * capturing stream returns DNNS_ERR_UNSUPPORTED and enqueues nothing.  All calls on a device share the one array and each call
 * clears the parts it needs at its start: calls that overlap on the GPU (different streams
 * without ordering between them) race on it and give wrong results; order them on one stream.
 */
#define DNNS_STATIC_MAX_NUMEL (1ull << 26)
dnns_status dnns_magnitude_threshold_static(const void* weights_dev, int32_t dtype, uint64_t numel, uint64_t k,
                                            dnns_threshold* thr_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DNNS_H */
