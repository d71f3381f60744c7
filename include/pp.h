/*
 * pp.h -- C interface of the pivoted (PBP) fully-connected inference library
 * for NVIDIA B200 (sm_100a).
 *
 * A layer computes  y = act(W x + b)  where the pruned matrix is in the
 * permutation-block-permutation form of Eq. 1,
 *
 *        W = P_row * W_piv * P_col ,
 *
 * W_piv holding only dense B x B tiles.  Evaluation follows Eq. 2 / Listing 1:
 * gather x through the column index array, multiply the kept tiles, scatter
 * through the row index array -- all inside one kernel per layer.
 *
 * Index arrays (Section 4.1.4): both map a PIVOTED index to an ORIGINAL index,
 *        x_piv[j] = x[col_perm[j]]          (gather, Listing 1 step 4)
 *        y[row_perm[i]] = y_piv[i]          (scatter, Listing 1 step 9)
 * so W[row_perm[i]][col_perm[j]] = W_piv[i][j].  Sizes that are not multiples
 * of B are padded in pivoted space: Mb = ceil(M/B), M_pad = Mb*B (same for N);
 * row_perm / col_perm are bijections on [0,M_pad) / [0,N_pad); pivoted rows
 * with row_perm[i] >= M are never stored and pivoted columns with
 * col_perm[j] >= N read x as 0.
 *
 * Pointer kinds: "host" = ordinary CPU memory, "device" = memory of the
 * current CUDA device.  All *_create calls copy what they are given; the caller
 * keeps ownership of its arrays.  Handles own their device memory until the
 * matching *_destroy.  The forward calls only ENQUEUE work on the given stream:
 * they never synchronise and never allocate (pp_forward_host, which works on
 * host buffers, is the one exception and says so below).  Calls that use the same handle
 * must be ordered on one stream (a handle owns scratch memory that concurrent
 * calls would share).  Every failure is a return code; nothing aborts or traps.
 * There is no CPU fallback.
 */
#ifndef PP_H_
#define PP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pp_layer pp_layer_t;
typedef struct pp_chain pp_chain_t;
typedef struct pp_packed pp_packed_t;

typedef enum {
    PP_OK = 0,
    PP_ERR_INVALID_ARG = 1, /* NULL pointer, non-positive size, misaligned device pointer, batch < 1 */
    PP_ERR_BAD_PERM = 2,    /* row_perm / col_perm is not a bijection on its padded range */
    PP_ERR_BAD_TILE = 3,    /* tile outside the Mb x Nb grid, or listed twice */
    PP_ERR_ALLOC = 4,       /* host or device allocation failed */
    PP_ERR_CUDA = 5,        /* a CUDA runtime call failed (no device, launch error, ...) */
    PP_ERR_UNSUPPORTED = 6, /* tile size / dtype / batch combination not implemented */
    PP_ERR_TIMEOUT = 7      /* a bounded device-side wait gave up (status word set by the kernel) */
} pp_status_t;

typedef enum { PP_F32 = 0, PP_F16 = 1 } pp_dtype_t;
typedef enum { PP_ACT_IDENTITY = 0, PP_ACT_RELU = 1 } pp_act_t;

const char* pp_status_string(pp_status_t s);

/* ------------------------------------------------------------------------- *
 * Host-side packer ("network implementation time", Sections 2 and 4.1.1: the
 * blocks may be ordered arbitrarily and mapped to the physical layout that
 * suits the architecture).  Validates the layer, sorts the kept tiles by
 * (block-row, block-col) and builds the block-row-compressed layout the
 * kernels read:
 *   - row_ptr[Mb+1]: first kept tile of each block-row (tile units);
 *   - col_ptr[Mb+1] / tile_col[]: per-block-row tile-column index arrays, each
 *     padded with -1 to a multiple of 4 entries (16 bytes);
 *   - values: kept tiles of a block-row contiguous, re-ordered into 512-byte
 *     "fragments" so that one 128-bit load per lane of a warp is fully
 *     coalesced (fp32: lane = row, 4 consecutive columns; fp16: the register
 *     layout of a 16x16 matrix-multiply operand);
 *   - gather_idx[N_pad] = col_perm with entries >= N replaced by -1,
 *     scatter_idx[M_pad] = row_perm with entries >= M replaced by -1,
 *     bias_piv[M_pad] = bias[row_perm[i]] (0 for padded rows or bias == NULL);
 *   - a work list cutting each block-row into parts of a few tiles.
 * Host only; needs no GPU.
 *
 * M, N          logical output / input sizes (> 0)
 * B             tile edge: 16, 32 or 64 (others: PP_ERR_UNSUPPORTED)
 * row_perm      host, int32[M_pad]     col_perm   host, int32[N_pad]
 * tile_list     host, int32[T][2] = (block_row, block_col), any order
 * tile_values   host, [T][B][B] row-major inside a tile, W_piv coordinates,
 *               element type wdtype (PP_F32: float, PP_F16: IEEE binary16 bits);
 *               entries on padding rows (row_perm >= M) or padding columns
 *               (col_perm >= N) are not part of W and are stored as zero
 * bias          host, float[M] in ORIGINAL row order, or NULL
 * ------------------------------------------------------------------------- */
pp_status_t pp_pack_create(pp_packed_t** out, int M, int N, int B,
                           const int32_t* row_perm, const int32_t* col_perm,
                           const int32_t* tile_list, int64_t T,
                           const void* tile_values, pp_dtype_t wdtype,
                           const float* bias);
pp_status_t pp_pack_destroy(pp_packed_t* p);

/* Sizes of the packed arrays: out[0]=Mb, [1]=Nb, [2]=T, [3]=length of tile_col
 * (padded), [4]=number of work items, [5]=bytes of packed values,
 * [6]=max tiles in one work item, [7]=number of partial-sum slots,
 * [8]=S strips (row-groups of block-rows), [9]=F fragments (512-byte units of values),
 * [10]=CTAs of the persistent kernel's plan, [11]=its cross-CTA partial-sum slots,
 * [12]=steps of the clustered tile kernel's plan (0 unless fp16 with B = 64). */
pp_status_t pp_pack_info(const pp_packed_t* p, int64_t out[13]);

/* Copy one packed array to host memory `dst` of capacity `bytes`.
 * which: 0 row_ptr(int32[Mb+1]) 1 col_ptr(int32[Mb+1]) 2 tile_col(int32[])
 *        3 gather_idx(int32[N_pad]) 4 scatter_idx(int32[M_pad]) 5 bias_piv(float[M_pad])
 *        6 values (bytes) 7 work items (int32[n_items][8]) 8 inv_row_perm(int32[M_pad])
 *        9 strip_start(int32[S+1]) 10 xoff(int32[F]) 11 CTA ranges (int32[G][4] =
 *        p_begin,p_end,s_first,s_count) 12 strip info (int32[S][4] = first_cta,nparts,slot_base,0)
 *        13 steps of the clustered tile kernel (int32[steps][8] = tile-column, sorted-tile index for each
 *        of the group's 4 block-rows or -1, tiles in the step, position of the step's first tile in the
 *        step-ordered tile images, 0; groups of 4 block-rows one after the other, tile-columns ascending
 *        inside a group) 14 its step boundaries (int32[ceil(Mb/4)][5]: CTA r of a group's cluster owns
 *        steps [b[r], b[r+1])) 15 position of every sorted tile in the step-ordered images (int32[T]) */
pp_status_t pp_pack_get(const pp_packed_t* p, int which, void* dst, int64_t bytes);

/* Plan of the persistent tensor-core kernel (fp16, B = 64) for n_ctas CTAs: the steps of pp_pack_get(13) cut into
 * one contiguous range per CTA, balanced by bytes, and the units (part of one group of 4 block-rows that one CTA
 * computes) in (group, step) order.  units_out: int32[n_units][8] = first step, end step, group, position among
 * the group's units, units of the group, index of the group's first unit, 0, 0; cta_unit_out: int32[n_ctas + 1],
 * CTA c owns units cta_unit[c] .. cta_unit[c + 1].  With units_out == cta_unit_out == NULL only *n_units_out is
 * written.  Host only.  Errors: PP_ERR_UNSUPPORTED for other layers, PP_ERR_INVALID_ARG. */
pp_status_t pp_pack_tile_units(const pp_packed_t* p, int n_ctas, int32_t* units_out, int64_t capacity_units,
                               int64_t* n_units_out, int32_t* cta_unit_out);

/* Inverse of the value re-ordering: writes the sorted tile list (int32[T][2])
 * and the tiles in their original row-major form ([T][B][B], wdtype). */
pp_status_t pp_pack_unpack(const pp_packed_t* p, int32_t* tile_list_out, void* tile_values_out);

/* Cross-layer permutation fusion (Section 4.2.1): the row permutation of layer
 * A followed by the column permutation of the next layer B is one static
 * permutation.  q[j] = position, in A's pivoted output, of the value that B's
 * pivoted column j reads:  q[j] = inv_row_perm_A[col_perm_B[j]], or -1 when
 * col_perm_B[j] >= N_B (padding).  Requires N_B == M_A.  Host only.
 * row_perm_A: int32[M_pad_A]; col_perm_B: int32[N_pad_B]; q_out: int32[N_pad_B]. */
pp_status_t pp_fold_perm(const int32_t* row_perm_A, int M_A, int M_pad_A,
                         const int32_t* col_perm_B, int N_B, int N_pad_B,
                         int32_t* q_out);

/* ------------------------------------------------------------------------- *
 * Layer: pack (as above) and upload to the current CUDA device.
 * Same arguments as pp_pack_create.  Errors: as pp_pack_create, plus
 * PP_ERR_CUDA / PP_ERR_ALLOC when no device is usable or memory runs out.
 * ------------------------------------------------------------------------- */
pp_status_t pp_layer_create(pp_layer_t** out, int M, int N, int B,
                            const int32_t* row_perm, const int32_t* col_perm,
                            const int32_t* tile_list, int64_t T,
                            const void* tile_values, pp_dtype_t wdtype,
                            const float* bias);
pp_status_t pp_layer_destroy(pp_layer_t* layer);

/* ------------------------------------------------------------------------- *
 * Irregular block structure (Section 4.1.5: blocks of different sizes, given to
 * the kernel through a table of block shapes; blocks that share rows need one
 * more reduction step).  W_piv holds n_blocks dense rectangles of any height,
 * width and position instead of tiles on a B x B grid.  This includes the
 * geometry the paper measures (Section 5: a size x size matrix with 1/fill-in
 * square blocks of edge size * fill-in, one per block-row).
 *
 * The rectangles are laid over the grid of B x B tiles the kernels work on:
 * every tile a block touches is kept, tile elements no block covers are zero,
 * and the products of tiles that share a block-row add up, which is that
 * reduction step.  So blocks whose edges are multiples of B and that start on
 * multiples of B cost exactly their own bytes; other shapes are padded to the grid.
 *
 * blocks        host, int32[n_blocks][4] = (first pivoted row, first pivoted
 *               column, height, width); 0 <= row, row + height <= M_pad (same for
 *               columns); height, width > 0; no element in two blocks
 * block_values  host, the blocks' values one block after the other, each
 *               row-major height x width, element type wdtype
 * M, N, B, row_perm, col_perm, wdtype, bias   as pp_pack_create
 *
 * pp_blocks_to_tiles is the host-side conversion on its own: *T_out receives the
 * number of tiles touched; with tile_list_out == tile_values_out == NULL it only
 * counts, otherwise it writes the tiles sorted by (block-row, block-column) into
 * tile_list_out (int32[T][2]) and tile_values_out ([T][B][B], wdtype), which
 * must hold capacity_tiles >= T tiles.  pp_pack_create_blocks and
 * pp_layer_create_blocks convert and then behave as pp_pack_create /
 * pp_layer_create.  Errors: PP_ERR_BAD_TILE for a block outside the padded
 * matrix, of non-positive size, or overlapping another; else as pp_pack_create.
 * ------------------------------------------------------------------------- */
pp_status_t pp_blocks_to_tiles(int M, int N, int B, const int32_t* blocks, int64_t n_blocks,
                               const void* block_values, pp_dtype_t wdtype, int64_t* T_out,
                               int32_t* tile_list_out, void* tile_values_out, int64_t capacity_tiles);
pp_status_t pp_pack_create_blocks(pp_packed_t** out, int M, int N, int B,
                                  const int32_t* row_perm, const int32_t* col_perm,
                                  const int32_t* blocks, int64_t n_blocks,
                                  const void* block_values, pp_dtype_t wdtype,
                                  const float* bias);
pp_status_t pp_layer_create_blocks(pp_layer_t** out, int M, int N, int B,
                                   const int32_t* row_perm, const int32_t* col_perm,
                                   const int32_t* blocks, int64_t n_blocks,
                                   const void* block_values, pp_dtype_t wdtype,
                                   const float* bias);

/* Raised by a kernel whose bounded device-side wait gave up (the call's output is then invalid).
 * Synchronises with the device; *status is PP_OK or PP_ERR_TIMEOUT.  The flag is cleared by the read. */
pp_status_t pp_layer_status(pp_layer_t* layer, pp_status_t* status);

/* Which kernel a pp_forward call with this batch launches, and its launch shape (for reports; host only):
 * out[0] kernel: 0 chunked matrix-vector, 1 persistent matrix-vector, 2 tensor-core tile kernel with one block-row
 * per CTA, 3 clustered tensor-core tile kernel, 4 persistent tensor-core tile kernel; out[1] CTAs; for the persistent kernel also out[2] asynchronous
 * weight copies each warp keeps in flight, out[3] bytes of dynamic shared memory per CTA, out[4] how x is staged
 * (StreamArgs::stage_mode), out[5] 1 when launched with programmatic stream serialization.  Assumes 16-byte
 * aligned x rows. */
pp_status_t pp_layer_launch_info(const pp_layer_t* layer, int batch, int32_t out[6]);

/* Independent device copy of a layer (own weights, index arrays and scratch), e.g. to
 * serve several streams at once or to rotate copies so that repeated timing runs do not
 * find the weights in L2.  Errors: PP_ERR_INVALID_ARG, PP_ERR_ALLOC, PP_ERR_CUDA. */
pp_status_t pp_layer_clone(pp_layer_t** out, const pp_layer_t* src);

/* y = act(W x + b) (Eq. 2, Listing 1 with both permutations).
 * x   device, [batch][N] row-major, element type = the layer's wdtype, 16-byte aligned
 * y   device, [batch][M] row-major, float, must not alias x
 * batch >= 1.  batch <= 8 runs the persistent matrix-vector kernel; larger batches run it in
 * groups of 8 columns or the chunked kernel in groups of up to 32; fp16 layers with B = 64 and
 * batch >= 9 run a tensor-core tile kernel in chunks of 128 rows (such layers keep a second copy of their
 * tiles on the device for it, unless they were created with tuning key 9 = 0).
 * cuda_stream: a cudaStream_t (NULL = default stream).  Enqueues only. */
pp_status_t pp_forward(pp_layer_t* layer, const void* x, void* y, int batch,
                       pp_act_t act, void* cuda_stream);

/* The same product (Eq. 2) from HOST buffers: copies x to the device, runs pp_forward and copies y
 * back, all on the given stream, and returns after the stream has drained, so y_host is valid on
 * return.  Unlike the calls above this one synchronises, and its first call on a layer (or a call
 * with a larger batch than any before) allocates the layer's two staging buffers.
 * x_host  host, [batch][N] row-major, element type = the layer's wdtype.  Pageable memory works (copy-engine
 *         transfers).  When both buffers are page-locked and mapped into the device's address space
 *         (cudaHostAlloc, cudaHostRegister) the library moves them with two small kernels of its own instead,
 *         which takes less time per call than setting up two transfers.
 * y_host  host, float [batch][M]
 * Errors: as pp_forward, plus PP_ERR_ALLOC. */
pp_status_t pp_forward_host(pp_layer_t* layer, const void* x_host, float* y_host, int batch,
                            pp_act_t act, void* cuda_stream);

/* Output permutation elimination (Section 4.2.2): the same product, but the result stays in
 * the layer's pivoted row order -- the last index array of Listing 1 is dropped and the host
 * relabels the coordinates when it interprets the result (an argmax, a softmax).
 * y_piv  device, float [batch][M_pad] (M_pad = M rounded up to a multiple of B), 16-byte
 *        aligned: y_piv[b][i] = act(W x + b)[map[i]]; padding positions (map[i] < 0) hold 0
 * pp_layer_output_map writes that map to HOST memory map[M_pad]: the original output row of
 * every pivoted position, -1 for padding.  Other arguments and errors as pp_forward. */
pp_status_t pp_forward_pivoted(pp_layer_t* layer, const void* x, float* y_piv, int batch,
                               pp_act_t act, void* cuda_stream);
pp_status_t pp_layer_output_map(const pp_layer_t* layer, int32_t* map);

/* ------------------------------------------------------------------------- *
 * Chain of layers with folded permutations (Section 4.2.1): the row permutation
 * of a layer and the column permutation of the next one are folded into one
 * static map (pp_fold_perm), which the producer applies when it stores: its
 * output lands directly in the consumer's pivoted column order and the consumer
 * reads it without any index array; only the first gather and the last scatter
 * touch original order.  Layer l's output feeds
 * layer l+1 rounded (to nearest even) to layer l+1's element type.
 * layers[l+1].N must equal layers[l].M.  The chain references its layers: they
 * must outlive it.  Intermediate buffers are sized for max_batch at create.
 * x: device [batch][N_0] (dtype of layer 0); y: device float [batch][M_last].
 *
 * Cross-layer permutation elimination (Section 4.2.3): a link whose folded map is the
 * identity (the consumer's column permutation equals the producer's row permutation on the
 * real rows, equal padded lengths) uses no index array at all: the producer stores its
 * pivoted rows as they are.  pp_chain_link_info writes identity[l] = 1 for every layer
 * l >= 1 whose incoming link is of that kind (identity[0] = 0) to HOST memory
 * identity[n_layers]; tuning key 13 = 0 sends such links through the map as well.
 *
 * Output permutation elimination (Section 4.2.2): after pp_chain_set_output_pivoted(chain, 1)
 * pp_chain_forward leaves y in the last layer's pivoted row order, float
 * [batch][M_pad_last], padding positions 0; pp_chain_output_map gives the relabelling
 * (as pp_layer_output_map of the last layer).  Errors: PP_ERR_INVALID_ARG.
 *
 * By default a chain is one kernel launch per layer, each launched with programmatic stream serialization so
 * that its prologue overlaps the previous layer's tail.
 *
 * One kernel for the whole chain (tuning key 14 = 1, set before pp_chain_create): when every layer has fp16
 * weights, batch <= 8 and the largest layer plan is resident on the device at once, pp_chain_forward is ONE
 * cooperative kernel launch.  Every CTA runs its share of layer 0, then of layer 1, ...; between two layers the
 * grid meets at a counter in device memory, and each CTA requests the tables and first weights of the next
 * layer one layer ahead, into the other of two shared-memory regions.  It measured slower than the launch per
 * layer on the 9216-4096-4096-1000 stack (a layer boundary inside the kernel is four dependent round trips
 * to the L2: publish, observe, fetch x, exchange partial sums), so it is not the default.  The waits are
 * bounded: when one gives up, the kernel raises a status word and ends, y is invalid and pp_chain_status
 * reports PP_ERR_TIMEOUT.  pp_chain_status synchronises with the device, also collects the status words of
 * the chain's layers (layer-by-layer execution), writes PP_OK or PP_ERR_TIMEOUT to *status and clears them. */
pp_status_t pp_chain_create(pp_chain_t** out, pp_layer_t* const* layers,
                            const pp_act_t* acts, int n_layers, int max_batch);
pp_status_t pp_chain_destroy(pp_chain_t* chain);
pp_status_t pp_chain_set_output_pivoted(pp_chain_t* chain, int enable);
pp_status_t pp_chain_output_map(const pp_chain_t* chain, int32_t* map);
pp_status_t pp_chain_link_info(const pp_chain_t* chain, int32_t* identity);
pp_status_t pp_chain_forward(pp_chain_t* chain, const void* x, void* y, int batch,
                             void* cuda_stream);
pp_status_t pp_chain_status(pp_chain_t* chain, pp_status_t* status);

/* ------------------------------------------------------------------------- *
 * Recurrent use: one pivoted layer as the gate matrix of an LSTM cell.  The
 * paper names recurrent networks only as users of FC layers; the cell below is
 * the usual one.  With z_t = [x_t ; h_{t-1}] (I + H entries) and g = W z_t
 * (4H rows, original order: [0,H) input gate i, [H,2H) forget gate f, [2H,3H)
 * candidate g, [3H,4H) output gate o; a bias given to the layer is part of g):
 *     c_t = sig(f) c_{t-1} + sig(i) tanh(g),     h_t = sig(o) tanh(c_t).
 * Following Section 4.2.1 the recurrence keeps z in the layer's pivoted column
 * order for all steps: the matrix-vector kernel reads it without a gather and
 * the gate kernel writes h_t straight to the pivoted positions step t+1 reads.
 * gates: a layer with M = 4H, N = I + H; it must outlive the handle.  Buffers
 * for max_steps steps are allocated at create.
 * x_seq  device, [steps][I], element type of the layer, 16-byte aligned
 * h      device, [H], element type of the layer: in h_0, out h_T (h is stored
 *        rounded to that type after every step, because it is a layer input)
 * c      device, float[H]: in c_0, out c_T
 * Enqueues work on the stream without synchronising.  fp16 gate layers whose
 * weights fit the shared memory of the whole GPU (one CTA per SM, H <= 2048)
 * run all steps in ONE cooperative kernel that keeps the weights on chip and
 * meets at one grid barrier per step (1 preparation kernel + 1 memset + 1
 * kernel; tuning key 11 = 0 switches this off); every other layer takes 1 + 2*steps
 * kernels.  The barrier's waits are bounded: when one gives up the kernel ends,
 * the outputs are invalid and pp_lstm_status reports PP_ERR_TIMEOUT.
 * pp_lstm_status synchronises with the device, writes PP_OK or PP_ERR_TIMEOUT
 * to *status and clears the flag. */
typedef struct pp_lstm pp_lstm_t;
pp_status_t pp_lstm_create(pp_lstm_t** out, pp_layer_t* gates, int I, int H, int max_steps);
pp_status_t pp_lstm_destroy(pp_lstm_t* lstm);
pp_status_t pp_lstm_forward(pp_lstm_t* lstm, const void* x_seq, void* h, float* c, int steps,
                            void* cuda_stream);
pp_status_t pp_lstm_status(pp_lstm_t* lstm, pp_status_t* status);

/* ------------------------------------------------------------------------- *
 * Feed-back search for the index arrays (Section 3.2: after training without
 * pruning, pick the permutations that keep the largest sum of absolute weights
 * in the upper-left and lower-right sub-blocks, by greedy optimisation from
 * given starting permutations; delete the off-diagonal half; repeat on every
 * remaining block, the number of blocks doubling each time).  Host only.
 *
 * The greedy step is read as an alternating balanced split: with the columns
 * fixed, the ceil(m/2) rows whose entries lean most to the first column half
 * take the first row half (the best balanced choice for those columns), then
 * the same for the columns with the rows fixed, until a sweep changes nothing
 * or max_sweeps is reached; ties go to the line that comes first; lines keep
 * their relative order inside a half.
 *
 * abs_w         host, float[M][N]: absolute values of the trained layer matrix
 * levels        bisections; the result has 2^levels diagonal blocks (fill-in
 *               2^-levels); needs 2^levels <= min(M, N)
 * row_init, col_init   host, int32[M] / int32[N]: starting permutations
 *               (pivoted -> original), NULL = identity
 * row_perm_out, col_perm_out   host, int32[M] / int32[N], pivoted -> original
 * blocks_out    host, int32[2^levels][4] = (first pivoted row, first pivoted
 *               column, height, width): the blocks pp_layer_create_blocks takes
 * kept_sum_out  host, sum of abs_w over the kept blocks; may be NULL
 * Errors: PP_ERR_INVALID_ARG, PP_ERR_BAD_PERM, PP_ERR_ALLOC.
 * ------------------------------------------------------------------------- */
pp_status_t pp_pivot_find(int M, int N, const float* abs_w, int levels, int max_sweeps,
                          const int32_t* row_init, const int32_t* col_init,
                          int32_t* row_perm_out, int32_t* col_perm_out, int32_t* blocks_out,
                          double* kept_sum_out);

/* ------------------------------------------------------------------------- *
 * Layout study (Section 4.1.1, Table 2): plain fp32 kernels over the three physical layouts of M_block the
 * paper compares, crossed with two ways of giving the work to threads.  They exist to repeat the paper's
 * comparison on this GPU and as the yardstick for the library's own kernels; no other call uses them.
 * Geometry of Section 5: a size x size matrix, n_blocks identical square blocks of edge size / n_blocks,
 * block k on pivoted rows and columns [k*edge, (k+1)*edge).  One input vector, no bias, no activation.
 *
 * layout: physical order of M_block (rightmost axis fastest):
 *   PP_LAYOUT_BRC block,row,column  PP_LAYOUT_BCR block,column,row  PP_LAYOUT_CBR column,block,row
 * mapping: PP_MAP_ROWS_PER_LANE   a lane owns one output row and walks along it (the thread mapping the
 *                                 paper describes: one thread per output coordinate);
 *          PP_MAP_LANES_ALONG_K   a warp owns four output rows, its lanes stride over the columns and
 *                                 the row sums are finished by a shuffle reduction.
 * row_perm, col_perm   host, int32[size], pivoted -> original (no padding)
 * block_values         host, float[n_blocks][edge][edge], row-major per block
 * x, y                 device, float[size]; must not alias
 * pp_layout_pack writes the values in the chosen layout to host memory out (n_blocks*edge*edge floats);
 * create uses it before the upload.
 * Errors: PP_ERR_INVALID_ARG (sizes, NULL, size not a multiple of n_blocks, unknown layout or mapping),
 * PP_ERR_BAD_PERM, PP_ERR_ALLOC, PP_ERR_CUDA.  pp_layout_forward only enqueues.
 * ------------------------------------------------------------------------- */
typedef struct pp_layout_study pp_layout_study_t;
typedef enum { PP_LAYOUT_BRC = 0, PP_LAYOUT_BCR = 1, PP_LAYOUT_CBR = 2 } pp_layout_t;
typedef enum { PP_MAP_ROWS_PER_LANE = 0, PP_MAP_LANES_ALONG_K = 1 } pp_mapping_t;
pp_status_t pp_layout_pack(int size, int n_blocks, pp_layout_t layout, const float* block_values, float* out);
pp_status_t pp_layout_create(pp_layout_study_t** out, int size, int n_blocks, pp_layout_t layout, pp_mapping_t mapping,
                             const int32_t* row_perm, const int32_t* col_perm, const float* block_values);
pp_status_t pp_layout_destroy(pp_layout_study_t* h);
pp_status_t pp_layout_forward(pp_layout_study_t* h, const float* x, float* y, void* cuda_stream);

/* ------------------------------------------------------------------------- *
 * Forward call that allocates nothing (the paper has no counterpart; this is a
 * packaging of pp_forward's small-batch kernel).
 *
 * For callers that may not allocate device memory where they run inference: a
 * real-time loop that owns one fixed arena, a process whose device memory pool
 * belongs to another runtime, a context in which cudaMalloc's implicit
 * synchronisation is forbidden.  Such a caller
 *   1. packs the layer on the host (pp_pack_create),
 *   2. asks for the size of the layer's device image (pp_pack_device_image_bytes),
 *      writes the image into host memory (pp_pack_device_image) and copies it to
 *      device memory it owns, 256-byte aligned,
 *   3. calls pp_forward_noalloc with that device pointer.
 * The scratch memory that CTAs sharing a strip of rows reduce through is a fixed
 * array of 1 MiB inside the library, resident on every GPU that loads it.
 * pp_forward_noalloc calls no cudaMalloc / cudaFree and no allocating routine.
 *
 * p             host, a packed layer; must stay alive while calls are in flight
 * device_image  device, the uploaded image of p (pp_pack_device_image), 256-byte aligned
 * x, y, act, cuda_stream   as pp_forward; batch must be 1..8
 * Errors: PP_ERR_UNSUPPORTED when batch > 8, when the layer's reduction scratch
 * (shared strips x rows x 8 floats, plus one counter per strip) exceeds the
 * 1 MiB array, when its plan has more than 320 CTAs or when x does not fit
 * shared memory; PP_ERR_INVALID_ARG for NULL / misaligned pointers;
 * PP_ERR_CUDA when a runtime call fails.
 * The first call on a device looks up the array's device address; make that call
 * before any stream capture.  All calls on a device share the array: it is re-
 * initialised by two memsets enqueued ahead of the kernel, and two calls that
 * overlap on the GPU (different streams) race on it.
 * pp_noalloc_status reports (and clears) the time-out flag of the current device's
 * pp_forward_noalloc kernels: *status is PP_ERR_TIMEOUT when a kernel's bounded wait
 * for the copy of x gave up since the last query (that call's y is invalid), else
 * PP_OK.  It synchronises with the device and allocates nothing either. */
pp_status_t pp_pack_device_image_bytes(const pp_packed_t* p, int64_t* bytes);
pp_status_t pp_pack_device_image(const pp_packed_t* p, void* host_dst, int64_t bytes);
pp_status_t pp_forward_noalloc(const pp_packed_t* p, const void* device_image,
                               const void* x, void* y, int batch, pp_act_t act,
                               void* cuda_stream);
pp_status_t pp_noalloc_status(pp_status_t* status);

/* Self-check of host-side bookkeeping that needs no GPU (the table that remembers, per device, which kernels
 * already have their shared-memory opt-in): PP_OK, or PP_ERR_INVALID_ARG when a check fails.  One process may
 * drive several GPUs; every kernel attribute is set once per device. */
pp_status_t pp_selftest_host(void);

/* Tuning knobs read at pack / create time (process-wide; for experiments).
 * key 0: target kilobytes of tile values per work item (default 32)
 * key 1: lower bound on the number of work items the splitter aims for (default 296)
 * key 2: CTAs of the persistent kernel (default 296)
 * key 3: minimum fragments per CTA of the persistent kernel (default 128)
 * key 4: -1 (default) lets the packer choose the persistent kernel's partition; 0..100 forces an even split
 *        over `key 2` CTAs (at least `key 3` fragments each) whose boundaries move onto a strip boundary when
 *        closer to it than this percentage of a CTA's share
 * key 5: 0 = never use the persistent kernel, 1 = use it when batch <= 8 and x fits shared memory (default 1)
 * key 6: asynchronous 512-byte weight copies each warp of the persistent kernel keeps in flight: 4, 6 or 8;
 *        0 (default) = with two CTAs per SM 4, or 8 for fp16 layers whose warps stream 17 fragments or more while
 *        two such CTAs still fit an SM; with one CTA per SM the deepest ring that fits
 * key 7: how the persistent kernel applies the column permutation: 2 (default) reads x through the index
 *        array inside the multiply loop for one input vector and, in fp16 layers, for 2..8 vectors; 1 does so
 *        for one vector only; 0 always permutes x into pivoted order in shared memory first
 * key 8: 1 (default) launches the persistent kernel with programmatic stream serialization, 0 plainly
 * key 10: 1 (default) permutes multi-column inputs in a pre-pass kernel when the layer kernel cannot hold x
 *         twice in shared memory; 0 leaves the gather to the layer kernel; 2 always uses the pre-pass
 * key 9: smallest batch for which fp16 layers with B = 64 take the tensor-core tile path (default 9: measured
 *        faster than the matrix-vector kernels from there on; 0 = never).  Such layers hold their tiles twice on
 *        the device (fragment order for the matrix-vector kernels, 8 KiB shared-memory images for the tile
 *        kernels: 2 x T x 8 KiB); a layer created while this key is 0 skips the second copy and never takes the
 *        tile path, whatever the key says later
 * key 12: tensor-core kernel of batched fp16 B = 64 layers: 0 or 1 (default) one block-row per CTA, its tiles
 *         dealt round robin to four warps that issue the tensor-core instructions into accumulators of their own
 *         (measured the fastest at every density and batch); 2 the clustered kernel (4 block-rows per cluster of
 *         4 CTAs share every X block); 3 the persistent kernel (one CTA per SM over an equal share of the layer's
 *         steps, two accumulator sets in tensor memory, groups split between CTAs summed through partial-sum
 *         slots in global memory in a fixed order: the key must be 3 when the layer is created, because the plan
 *         and its slots, 128 KiB per unit, are only allocated then; other layers fall back to one block-row per
 *         CTA).  2 and 3 are kept as options
 * key 13: 1 (default) chain links whose folded map is the identity store pivoted rows without an index array,
 *         0 sends them through the map like any other link
 * key 11: 1 (default) lets pp_lstm_forward run all steps in one cooperative kernel when the layer qualifies, 0 never
 * key 14: 1 chains of fp16 layers run as one cooperative kernel when they qualify (read at pp_chain_create
 *         and at every pp_chain_forward), 0 (default) one launch per layer
 * key 15: polls after which the bounded device-side waits of the persistent kernel (copy of x) and of the chain
 *         kernel (layer boundaries) give up; 0 (default) = the kernels' own limits (seconds).  Small values exist
 *         so that tests can see a wait give up: the kernel then raises its status word and still ends by itself
 * key 16: 1 (default) pp_forward_host moves page-locked host buffers that the device can address with small
 *         kernels, 0 always uses cudaMemcpyAsync
 * key 17: 1 is the caller's promise, for the pp_forward / pp_forward_pivoted calls made while it is set, that x was
 *         complete before any kernel still in flight in the stream was enqueued (independent requests whose inputs
 *         were uploaded earlier; NOT a chain, where x is the previous call's y).  The persistent kernel (batch <= 8)
 *         then fetches x before it waits for the previous kernel and waits only in front of its first write to y
 *         or scratch, so consecutive calls overlap further; other kernels ignore the key.  0 (default): every read
 *         of x waits for the previous kernel.  With the promise broken the call reads x too early: wrong values,
 *         no fault */
pp_status_t pp_set_tuning(int key, int value);

#ifdef __cplusplus
}
#endif
#endif /* PP_H_ */
