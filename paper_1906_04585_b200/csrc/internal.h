// Internal declarations shared by the CUDA sources of the GALA learner library.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "gala.h"

namespace gala {

// ---------------------------------------------------------------- programmatic dependent launch
// Kernels of the learner step are launched so that a kernel may become resident while its predecessor
// in the stream is still running.  A kernel first does the set-up that touches no data of the step
// (barriers, tensor memory, descriptor prefetch), then waits for the predecessor to complete and its
// writes to be visible (pdl_wait), then lets its own successor start (pdl_launch).  Because the trigger
// comes after the wait, at most two consecutive kernels overlap: what a kernel reads before pdl_wait
// must have been written at least two kernels earlier.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ---------------------------------------------------------------- network layout
// Offsets (in floats) of every tensor inside one agent's flat vector.
struct ConvLayout {
    long w[3], b[3];      // conv1..3
    long fcw, fcb;        // hidden layer 3136 -> 512
    long piw, pib, vw, vb;
};
struct MlpLayout {
    long w1, b1, w2, b2;
    long piw, pib, vw, vb;
};

// Fixed geometry of the conv trunk (Appendix C.2 network at 84x84x4).
constexpr int kFrameH = 84, kFrameW = 84, kFrameC = 4;
constexpr int kConvK[3] = {8, 4, 3};
constexpr int kConvS[3] = {4, 2, 1};
constexpr int kConvCin[3] = {4, 32, 64};
constexpr int kConvCout[3] = {32, 64, 64};
constexpr int kConvIn[3] = {84, 20, 9};    // input height = width
constexpr int kConvOut[3] = {20, 9, 7};    // output height = width
constexpr int kConvKK[3] = {256, 512, 576};  // k*k*cin
constexpr int kFeat = 3136, kHidden = 512;

// Caller-owned per-agent pointers travel in kernel parameters, at most kBatch agents a launch.
constexpr int kBatch = 64;
struct PtrBatch { const void* p[kBatch]; };

// Which agents a launch works on.  Group gz of a launch (0 .. groups - 1) addresses the per-agent tensors of the
// library (parameters, gradients, workspaces) as agent slot(gz): gz itself for the consecutive agents
// [agent0, agent0 + groups) - every base pointer is then already moved to agent0 - or entry gz of a list of agent
// indices (base pointers are agent 0's).  Pointers that come with the launch (PtrBatch) are always indexed by gz.
struct AgentMap {
    int on;
    unsigned char v[kBatch];
};
__host__ __device__ __forceinline__ int agent_slot(const AgentMap& m, int gz) { return m.on ? (int)m.v[gz] : gz; }

// ---------------------------------------------------------------- GEMM
// One operand of the grouped tensor-core GEMM, as a TMA descriptor plus what
// the kernel must know about its shared-memory image.
struct GemmOperand {
    CUtensorMap map;
    int mn_major;  // 0: stored [rows = M or N][K]; 1: stored [K][M or N]
};

enum EpilogueFlags : int {
    EPI_OUT_BF16 = 1,    // store bf16 (else fp32)
    EPI_RELU = 2,        // max(.,0) after scale and bias
    EPI_TRANSPOSE = 4,   // store D[m][n] at out[n*ldc + m]
    EPI_MASK = 8,        // multiply by (mask[m][n] > 0), mask bf16 with the output's layout
    EPI_GATE = 32,       // zero where bit n % 32 of gate[m][n / 32] is clear (ReLU gate bits; N a multiple of 32)
    EPI_ROWMAP_S2 = 16   // rows are (sample, parity class, a, c) of a stride-2 data gradient: row r of tile
                         // (sample, class) goes to pixel (2a + class/2, 2c + class%2) of the 20x20 input grid
};

struct GemmArgs {
    int M, N, K;           // valid extents of one group's product
    int block_n;           // 32, 64 or 128
    int groups;            // grid.z = groups * split_k
    int group0;            // first group index (added to the TMA group coordinate)
    int split_k;
    int stages;            // shared-memory ring depth; set by launch_gemm
    int flags;
    float scale;           // applied to the accumulator before the bias
    const float* bias;     // per-column (n) bias, may be null; indexed by group with bias_group_stride
    long bias_group_stride;
    void* out;             // group g, split s at out + g*out_group_stride + s*out_split_stride (elements)
    long out_group_stride;
    long out_split_stride;
    long ldc;
    const __nv_bfloat16* mask;  // [m][n] with the output's ldc; group g at mask + g*mask_group_stride
    long mask_group_stride;
    const uint32_t* gate;       // [m][N / 32] words; group g at gate + g*gate_group_stride
    long gate_group_stride;
    int* error_word;       // device int, set non-zero when a bounded wait runs out
    int max_ctas;          // > 0: at most this many CTAs (leaves SMs to kernels of other streams)
    AgentMap am;           // agents behind the groups (operands, outputs, bias, mask, gate, sq_partial)
    // Optional sums of squares of the stored outputs (for a gradient norm without a second pass over this
    // product): slot [tile * (block_n / 8) + warp quarter * (block_n / 32) + 32-column block] of sq_partial gets the sum over that
    // 32 x 32 block (0 where the block lies outside the matrix).  Needs block_n = 128, split_k = 1, fp32 row-major
    // output with 32-byte aligned rows and N a multiple of 32; tile = (group * m_tiles + m_tile) * n_tiles + n_tile.
    float* sq_partial;
    // Tiling (set by the caller for the convolution modes, filled with defaults by launch_gemm)
    int tile_rows;         // rows of D per M tile (<= 128; default 128)
    int k_steps;           // number of K steps of the whole reduction (default ceil(K/64))
    // Implicit convolution operands (conv_mode != CONV_NONE): the patch matrix is never stored; TMA
    // boxes over the NHWC activations deliver, for one kernel offset, the [patch][channel] block.
    int conv_mode;
    int conv_layer;        // 0: conv1 (8x8 stride 4 on bf16 copies of the 84x84x4 frames), 1: conv2 (4x4 stride 2
                           // on 20x20x32), 2: conv3 (3x3 stride 1 on 9x9x64)
    int conv_nb;           // samples per M tile (forward, data gradient) or per K step (weight gradient)
    int a_samples;         // samples per group in the activation tensor behind A
    int b_samples;         // weight gradient: samples per group in the dY tensor behind B
    int kstep_rows;        // weight gradient: rows of a K step in shared memory (multiple of 16)
    int box_rows;          // rows of one A box (patches or pixels it delivers)
    int kpack;             // forward / data gradient: kernel-offset blocks (A box + B box each) per K step
    int conv_q;            // number of such blocks in the whole reduction (set by launch_gemm)
    int a_sub_bytes;       // distance between the A boxes of one K step (set by launch_gemm)
    int stage_a_bytes, stage_b_bytes;   // set by launch_gemm
};
//   CONV_FWD  : D[patch][co]  = sum_k patches[patch][k] W[co][k]      A from boxes, B = weights (K-major)
//   CONV_WGRAD: D[k][co]      = sum_patch patches[patch][k] dY[patch][co]   A (transposed patches) and B from boxes
//   CONV_DGRAD: dX[pixel][ci] = sum_{offset, co} dY[pixel - offset][co] W[co][offset][ci]; A = boxes of dY shifted
//               by the kernel offset (out-of-range entries read as zero), B = the offset's [co][ci] block of W
enum ConvMode : int { CONV_NONE = 0, CONV_FWD = 1, CONV_WGRAD = 2, CONV_DGRAD = 3 };

cudaError_t gemm_init();   // resolves the driver entry point used to build TMA descriptors
// Streaming multiprocessors of the current device (asked once per device; 148 if the query fails): what grids and
// slice counts are sized by.
int sm_count();
// rows x cols bf16 matrix per group, cols contiguous.  box_rows x box_cols tile.
bool make_tensor_map(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t groups,
                     uint64_t row_stride_bytes, uint64_t group_stride_bytes, uint32_t box_cols,
                     uint32_t box_rows);
// rows x cols fp32 matrix, unswizzled box_rows x box_cols tile (gemm_init() first).
bool make_tensor_map_f32(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes,
                         uint32_t box_cols, uint32_t box_rows);
bool make_tensor_map_f32_wide(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes,
                              uint32_t box_blocks, uint32_t box_rows);
// General bf16 tensor map of rank 3..5 (dims/strides innermost first).  swizzle: 0 = 128-byte, 1 = 64-byte
// (64-byte rows), 2 = 32-byte (32-byte rows), 3 = none.  Dimensions may overlap (a stride smaller than the extent
// below it); a box may be larger than a dimension (the rest reads as zero).
bool make_tensor_map_nd(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                        const uint64_t* strides_bytes, const uint32_t* box, int swizzle = 0);
// Builds the descriptor for an operand of a GEMM with the given tile height
// (128 for A, block_n for B).
bool make_operand(GemmOperand* op, const void* base, int mn_major, uint64_t mn_extent, uint64_t k_extent,
                  uint64_t groups, uint64_t ld_elems, uint64_t group_stride_elems, int tile_mn);
cudaError_t launch_gemm(const GemmOperand& A, const GemmOperand& B, const GemmArgs& args, cudaStream_t st);
cudaError_t launch_splitk_reduce_act(const float* partials, __nv_bfloat16* out, const float* bias, long bias_group_stride,
                                     int group0, long count, int N, int split_k, long split_stride, int groups,
                                     long partial_group_stride, long out_group_stride, cudaStream_t st);
cudaError_t launch_splitk_reduce(const float* partials, float* out, long count, int split_k,
                                 long split_stride, int groups, long partial_group_stride,
                                 long out_group_stride, cudaStream_t st);

// Several sliced weight (and bias) gradients finished in one launch: range k of the output (out_off, count floats) is the sum,
// in slice order, of `split` slices that lie `count` floats apart from ws_off on in the group's workspace.  Offsets
// and counts are multiples of 4 floats.
struct ReduceSeg { long out_off, count, ws_off; int split; };
struct ReduceSegs { ReduceSeg s[6]; int n; };
cudaError_t launch_splitk_reduce_multi(const float* ws, float* out, const ReduceSegs& segs, int groups,
                                       long ws_group_stride, long out_group_stride, cudaStream_t st,
                                       const AgentMap* am = nullptr);

// ---------------------------------------------------------------- convolutions with a resident input
// Forward and data-gradient convolutions of the trunk (conv.cu).  Tensors are NHWC bf16; weights
// W[co][(ky, kx, ci)] bf16; group g (agent) uses sample block g * a_samples.. of the input tensor.
enum ConvVariant : int { CV_CONV1_FWD = 0, CV_CONV2_FWD, CV_CONV3_FWD, CV_CONV2_DGRAD, CV_CONV3_DGRAD };
struct ConvArgs {
    int variant;
    int groups, group0;    // agents of this launch: group0 .. group0 + groups - 1
    int rows;              // samples per agent to process
    int a_samples;         // samples per agent in the input tensor
    float scale;           // forward: applied to the accumulator before the bias
    const float* bias;     // forward: per output channel, agent g at bias + g * bias_group_stride
    long bias_group_stride;
    __nv_bfloat16* out;    // first agent of the launch; agent i of the launch at out + i * out_group_stride
    long out_group_stride;
    // ReLU gates, one bit per channel and pixel: word [sample][pixel][channel / 32], bit channel % 32 set
    // when the stored activation is positive.  Forward (conv1, conv2): written next to the activation
    // (may be null); data gradient: the gates of the layer input, which multiply the result.
    uint32_t* gate_out;
    const uint32_t* gate_in;
    long gate_group_stride;      // words per agent
    int* error_word;
    int max_ctas;          // > 0: at most this many CTAs (leaves SMs to kernels of other streams)
    AgentMap am;           // agents behind the groups
    PtrBatch obs;          // conv1 forward: the agents' uint8 frames [rows][84][84][4], 16-byte aligned
    // conv2 data gradient (may be null): per-channel sums over the pixels of the result, as slices
    // [agent of the launch][kConvMaxGrid CTAs][8 warps][32 channels].  CTA b (of `grid`) works on samples
    // [total * b / grid, total * (b + 1) / grid) of the launch's groups * rows and writes the slices of every agent
    // that range touches; the other slices are left alone and must not be read.
    float* bias_partial;
};
constexpr int kConvMaxGrid = 148;   // most CTAs a convolution launch uses (the bias slices are laid out for it)
constexpr long kConvBiasSliceStride = (long)kConvMaxGrid * 8 * 32;   // floats per agent
int conv_grid(long units, int max_ctas);   // CTAs of a launch over `units` work units
cudaError_t conv_init();
bool make_conv_maps(int variant, CUtensorMap* x_map, CUtensorMap* w_map, const void* x_base, uint64_t samples,
                    const void* w_base, uint64_t groups, uint64_t w_group_stride_elems);
cudaError_t launch_conv(const CUtensorMap& x, const CUtensorMap& w, const ConvArgs& a, cudaStream_t st);

// ---------------------------------------------------------------- conv weight gradients, resident operands
// conv2 / conv3 weight gradients (wgrad.cu): x = the layer's input activation, y = dY of the layer.
enum WgradVariant : int { WG_CONV2 = 1, WG_CONV3 = 2 };
struct WgradArgs {
    int variant;
    int groups, group0;    // agents of this launch
    int splits;            // CTAs per agent, each takes a slice of the samples
    int samples;           // samples per agent to reduce over
    int x_samples, y_samples;   // samples per agent in the two tensors
    float* out;            // agent i, slice s at out + i * out_group_stride + s * out_split_stride, as W[co][KK]
    long out_group_stride, out_split_stride;
    // bias gradient (column sums of dY over the same samples), summed from the dY tiles while they are in shared
    // memory: agent i, slice s at bias_out + i * bias_group_stride + s * bias_split_stride, 64 floats; null: not wanted
    float* bias_out;
    long bias_group_stride, bias_split_stride;
    int* error_word;
    AgentMap am;           // agents behind the groups
};
cudaError_t wgrad_init();
bool make_wgrad_maps(int variant, CUtensorMap* x_map, CUtensorMap* y_map, const void* x_base, uint64_t x_samples,
                     const void* y_base, uint64_t y_samples);
cudaError_t launch_wgrad(const CUtensorMap& x, const CUtensorMap& y, const WgradArgs& a, cudaStream_t st);

// conv1 weight gradient from the uint8 frames (wgrad1.cu); y = dY of conv1 [sample][20][20][32] bf16
struct Wgrad1Args {
    int groups, group0;    // agents of this launch
    int splits;            // CTAs per agent, each takes a slice of the samples
    int samples;           // samples per agent to reduce over (the first `samples` frames of each agent)
    int y_samples;         // samples per agent in the dY tensor
    float scale;           // applied to the sums (1/255: the frames enter the network divided by 255)
    float* out;            // agent i, slice s at out + i * out_group_stride + s * out_split_stride, as W[32][256]
    long out_group_stride, out_split_stride;
    int* error_word;
    AgentMap am;           // agents behind the groups
    PtrBatch obs;          // the agents' uint8 frames [..][84][84][4], 16-byte aligned
};
cudaError_t wgrad1_init();
bool make_wgrad1_map(CUtensorMap* y_map, const void* y_base, uint64_t y_samples);
cudaError_t launch_wgrad1(const CUtensorMap& y, const Wgrad1Args& a, cudaStream_t st);

// ---------------------------------------------------------------- sweep
struct SweepHp {
    float lr, alpha, eps;
};
// Per-agent asynchronous form.  Any of peer0/peer1 may be null (n_peers says how many are used).
cudaError_t launch_sweep_agent(float* x, const float* g, float* v, float* snap_out, const float* peer0,
                               const float* peer1, int n_peers, const float* clip, __nv_bfloat16* shadow,
                               long d_pad, SweepHp hp, cudaStream_t st);
// Per-agent form for up to kBatch agents in one launch (sweep_many.cu).  Rows are indices into row-major arrays of
// d_pad floats: x_row into x, g, v, clip and shadow (the agent), out_row and p_row into `snap` (agent * slots + slot).
// No out_row of a launch may equal a p_row of the same launch.
struct SweepItem {
    int x_row;
    int out_row;      // where y, the agent's new snapshot, goes
    int p_row[2];     // snapshots averaged with y (-1: none; p_row[1] only with p_row[0])
};
struct SweepManyArgs {
    float* x; const float* g; float* v; float* snap;
    __nv_bfloat16* shadow;      // optional bf16 copy of the new x
    const float* clip;          // per agent, or null (= 1)
    long d_pad;
    SweepHp hp;
    int* error_word;
    int n_items;
    int max_ctas;               // > 0: at most this many CTAs
    int rows, cols, stages;     // set by the launcher
    unsigned has_grad[kBatch / 32];   // bit e: item e applies a pending gradient (else y = x, v untouched)
    SweepItem it[kBatch];
};
cudaError_t launch_sweep_many(const SweepManyArgs& a, cudaStream_t st);
// Synchronous all-agent form.  peer_off[j]: in-peer j of agent i is (i - peer_off[j]) mod n.
cudaError_t launch_sweep_sync(float* x, const float* g, float* v, const float* clip,
                              __nv_bfloat16* shadow, int n_agents, long d_pad, int n_peers,
                              const int* peer_off, SweepHp hp, int* error_word, cudaStream_t st);
// Bulk-copy staged variant; cudaErrorNotSupported when the shape does not suit it.
cudaError_t launch_sweep_sync_bulk(float* x, const float* g, float* v, const float* clip, __nv_bfloat16* shadow,
                                   int n_agents, long d_pad, int n_peers, int o0, int o1, SweepHp hp,
                                   int* error_word, cudaStream_t st);
// Sum of squares of g[agent][0..d) -> norm[agent], clip[agent] = min(1, max_norm/(norm+1e-6)).
// partial: [n_agents][kNormChunks] doubles, ticket: [n_agents] uints (zero before first use).
constexpr int kNormChunks = 128;
// A range of g whose sum of squares is already known as partial sums (written by the product that produced it):
// the norm pass skips reading it and adds the partials in slot order instead.
struct NormKnown { long off, count; const float* partial; long n_partials, partial_group_stride; };
cudaError_t launch_grad_norm(const float* g, long d, long d_pad, int agent0, int n_agents, float max_norm,
                             double* partial, unsigned* ticket, float* norm, float* clip, cudaStream_t st,
                             const NormKnown* known = nullptr, const AgentMap* am = nullptr);
cudaError_t launch_allreduce_grads(float* g, int n_agents, long d_pad, cudaStream_t st);
// partial: 592 doubles, ticket: one zeroed unsigned, out: one double (squared distance)
// ||alpha G||_F^2 of the coming optimiser pass (see update_norm_kernel).  partial: [n_agents][kUpdateNormChunks]
// doubles, ticket: one uint (zero before first use), out: one double.
constexpr int kUpdateNormChunks = 32;
cudaError_t launch_update_norm(const float* g, const float* v, const float* clip, int n_agents, long d_pad, SweepHp hp,
                               double* partial, unsigned* ticket, double* out, cudaStream_t st);
cudaError_t launch_consensus(const float* x, int n_agents, long d, long d_pad, double* partial, unsigned* ticket,
                             double* out, cudaStream_t st);
cudaError_t launch_delay(unsigned long long usec, cudaStream_t st);
cudaError_t launch_wait_runs_out(unsigned polls, int* error_word, cudaStream_t st);
cudaError_t launch_cast_bf16(const float* x, __nv_bfloat16* out, long count, cudaStream_t st);

// ---------------------------------------------------------------- A2C pieces

struct LossArgs {
    int T, E, A;
    float gamma, ent_coef, vf_coef;
    const float* logits;   // [agents][B][A]
    const float* values;   // [agents][B]
    PtrBatch actions, rewards, dones;  // per agent [T][E]
    float* returns;        // [agents][S]
    float* adv;            // [agents][S]
    float* dlogits;        // [agents][S][A]
    float* dvalues;        // [agents][S]
    float* losses;         // [agents][4]
    long B;                // (T+1)*E
};
cudaError_t launch_a2c_loss(const LossArgs& a, int n_agents, cudaStream_t st);
cudaError_t launch_sample(const float* logits, const float* uniforms, int* actions, int E, int A,
                          cudaStream_t st);

// Small dense layers on the CUDA cores (fp32 accumulate).  TIn: float or bf16.
// act: 0 none, 1 relu, 2 tanh.  Group g uses W + g*w_stride etc.
struct DenseArgs {
    int rows, in_dim, out_dim, act;
    PtrBatch in;                           // per group [rows][in_dim]
    int in_bf16;
    const float* W; const float* b; long w_stride;  // W[out][in], b[out] inside the flat vector
    void* out; long out_stride; int out_bf16;       // [g][rows][out_dim]
};
cudaError_t launch_dense_fwd(const DenseArgs& a, int groups, cudaStream_t st);
// heads: logits[g][rows][A], values[g][rows]
struct HeadsArgs {
    int rows, H, A;
    const void* h; long h_stride; int h_bf16;
    const float* params; long p_stride;   // flat vectors; offsets below
    long piw, pib, vw, vb;
    float* logits; long logits_stride;
    float* values; long values_stride;
};
cudaError_t launch_heads_fwd(const HeadsArgs& a, int groups, cudaStream_t st);
struct HeadsBwdArgs {
    int rows, H, A, act;   // rows = S; act of the hidden layer (1 relu, 2 tanh)
    const void* h; long h_stride; int h_bf16;
    const float* params; long p_stride;
    long piw, pib, vw, vb;
    const float* dlogits; long dlogits_stride;   // [g][S][A]
    const float* dvalues; long dvalues_stride;   // [g][S]
    const float* dzv;                            // optional [g][S][20]: rows (dlogits, dvalue, zeros), 16-byte aligned
    float* grad; long g_stride;                  // flat gradient (same offsets)
    void* dpre; long dpre_stride; int dpre_bf16; // [g][S][H] dL/d(pre-activation of hidden)
    AgentMap am;                                 // agents behind the groups (tiled weight-gradient kernel only)
};
// data part (dpre) and parameter part (gradients of the head weights and biases): independent of each other
cudaError_t launch_heads_dgrad(const HeadsBwdArgs& a, int groups, cudaStream_t st);
cudaError_t launch_heads_wgrad(const HeadsBwdArgs& a, int groups, cudaStream_t st);
// same sums with the samples split over the warps of a block per 32 columns (fixed order); not supported
// (cudaErrorNotSupported) for more than 18 actions or a width that is not a multiple of 32
cudaError_t launch_heads_wgrad_tiled(const HeadsBwdArgs& a, int groups, cudaStream_t st);
// Heads of the conv net (width 512, bf16 ReLU activations) fused with returns, advantages, objective and
// the gradient of the hidden pre-activation; see a2c.cu.
struct HeadsFusedArgs {
    int T, E, A;
    int ne;                 // environments per block (set by the launcher)
    float gamma, ent_coef, vf_coef;
    const __nv_bfloat16* hid;   // [g][B][512] stored activations (used when partials == null)
    __nv_bfloat16* hid_out;     // where the activations are stored when they are formed here
    long h_stride;
    const float* partials;      // optional split-K partial sums of the hidden layer [g][split][B][512]
    int split; long split_stride, partial_group_stride;
    const float* params; long p_stride;   // flat vectors of the first agent of the launch
    long piw, pib, vw, vb, fcb;
    PtrBatch actions, rewards, dones;     // per agent [T][E]
    float *logits, *values;               // [g][B][A], [g][B]
    float *returns, *adv, *dlogits, *dvalues;   // [g][S], [g][S], [g][S][A], [g][S]
    float* dzv;                           // [g][S][20]: rows (dlogits, dvalue, zeros) for the weight-gradient kernel
    float* losses;                        // [g][4]
    long B;                               // (T+1)*E
    __nv_bfloat16* dh; long dh_stride;    // [g][S][512]
    float* loss_partial;                  // [g][E][4] scratch
    unsigned* ticket;                     // [g], zero before the first launch
    AgentMap am;                          // agents behind the groups
};
bool heads_fused_supported(int T, int E, int A, int H);
int heads_fused_blocks(int T, int E, int groups);   // blocks per agent of a launch with `groups` agents
cudaError_t launch_heads_fused(const HeadsFusedArgs& a, int groups, cudaStream_t st);
struct DenseBwdArgs {
    int rows, in_dim, out_dim, act_in;    // act_in: activation that produced `in` (0 none: no dgrad)
    PtrBatch in;                          // per group [rows][in_dim]  (fp32)
    const float* dpre; long dpre_stride;  // [g][rows][out_dim]
    const float* W; long w_stride;        // flat params + offset of W
    float* gW; float* gb; long g_stride;  // flat grad + offsets
    float* din; long din_stride;          // [g][rows][in_dim] dL/d(pre-activation of previous layer); null: skip
};
cudaError_t launch_dense_bwd(const DenseBwdArgs& a, int groups, cudaStream_t st);

// ---------------------------------------------------------------- MLP learner step in one kernel (mlp_fused.cu)
struct MlpFusedArgs {
    int D, H, A, T, E;
    long d;                               // parameters per agent
    MlpLayout l;
    float gamma, ent_coef, vf_coef, max_norm;
    const float* params; long p_stride;   // first agent of the launch
    PtrBatch obs, actions, rewards, dones;
    float *logits, *values, *returns, *adv, *dlogits, *dvalues, *losses;   // first agent of the launch
    float *h1_out, *h2_out;               // [g][B][H] hidden activations
    float* grad; long g_stride;
    float *norm, *clip;                   // [g]
    float* partial;                       // [g][kMlpMaxBlocks][mlp_fused_partial_stride(d)] scratch
    unsigned* ticket;                     // [g], zero before the first launch
    int ne, nb_max; long partial_stride;  // set by the launcher
};
constexpr int kMlpMaxBlocks = 16;         // blocks per agent
long mlp_fused_partial_stride(long d);
bool mlp_fused_supported(int D, int H, int A, int T, int E, long d);
cudaError_t launch_mlp_fused(const MlpFusedArgs& a, int groups, cudaStream_t st);

// ---------------------------------------------------------------- synthetic environment (env.cu)
struct EnvArgs {
    unsigned long long seed;
    int agent, n_actions;
    const long long* step_base;  // device counter added to `step` and `obs_step` (null: they are absolute)
    long long step;              // transition whose reward / done flag is produced (if actions != null)
    const int* actions;          // [E] actions taken at `step`, or null
    float* rewards;              // [E]
    unsigned char* dones;        // [E]
    long long obs_step;          // step whose observation and action-draw uniform are produced (if obs_out != null)
    void* obs_out;               // [E][obs_elems] uint8 frames or float vectors, or null
    float* uniforms;             // [E]
    long obs_elems;              // bytes (frames) or floats (vectors) per environment
    int frames;                  // 1: uint8 frames, 0: float vectors
};
cudaError_t launch_env(const EnvArgs& a, int n_envs, cudaStream_t st);
// All agents of a lockstep loop in one launch (see env_act_all_kernel).
struct EnvActArgs {
    unsigned long long seed;
    int n_actions, draw, frames;
    const long long* step_base;  // [n] device counters, added to `step`
    long long step;              // draw: the transition taken; else the step whose observation is written
    const float* logits;         // agent i's logits of its E environments at logits + i * logits_stride
    long logits_stride;
    int* actions; float* rewards; unsigned char* dones;   // element (i, e) at i * te_stride + te_off + e
    long te_stride, te_off;
    void* obs_out;               // agent i's observations at obs_out + i * obs_agent_stride + obs_off (bytes)
    long obs_agent_stride, obs_off;
    long obs_elems;              // bytes (frames) or floats (vectors) per environment
    int agent0;                  // first agent of the launch (grid.z counts from it)
    // H > 0: the policy head is formed here from the hidden layer instead of read from `logits`: hidden unit u of
    // environment e = bf16(relu(sum over the splits of partials + bias)) if split > 0, else hid[e][u]
    int H, split;
    const float* partials; long split_stride, partial_group_stride;   // [i][split][E][H]
    const __nv_bfloat16* hid; long h_stride;                          // [i][.][H]
    const float* params; long p_stride;                               // flat parameter vectors, agent 0 first
    long piw, pib, fcb;
};
cudaError_t launch_env_act_all(const EnvActArgs& a, int n_envs, int n_agents, cudaStream_t st);
cudaError_t launch_env_advance_all(long long* counters, int n, long long by, cudaStream_t st);
cudaError_t launch_env_advance(long long* counter, long long by, cudaStream_t st);

// ---------------------------------------------------------------- conv lowering
// uint8 frames -> bf16 (exact), per group [samples][84*84*4]
cudaError_t launch_cast_frames(const PtrBatch& obs, __nv_bfloat16* out, long out_group_stride, int samples, int groups,
                               cudaStream_t st);
// Column sums (bias gradients) of up to kColsumJobs bf16 tensors in one launch:
// out_base[g*out_group_stride + out_off + c] = sum_r dy[g][r][c], fixed summation order.
// partial: [groups][kColsumJobs][kColsumChunks][512] doubles, ticket: [groups][kColsumJobs] (zeroed once).
constexpr int kColsumJobs = 4;
struct ColsumJob { const __nv_bfloat16* dy; long group_stride; long rows; int C; long out_off; };
struct ColsumJobs { ColsumJob j[kColsumJobs]; };
// slices: when slices.partial is set, one more block per agent adds the bias slices that a conv2 data-gradient
// launch of `grid` CTAs over groups * rows samples left behind (ConvArgs::bias_partial), in CTA and warp order,
// into out_base[g*out_group_stride + out_off + 0..31].
struct ColsumSlices { const float* partial; long out_off; int grid, rows; };
cudaError_t launch_colsum(const ColsumJobs& jobs, int n_jobs, float* out_base, long out_group_stride, double* partial,
                          unsigned* ticket, int groups, cudaStream_t st, const ColsumSlices* slices = nullptr,
                          const AgentMap* am = nullptr);
constexpr int kColsumChunks = 64;

}  // namespace gala
