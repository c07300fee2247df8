// C ABI of the GALA learner library: context, topology schedule, per-agent streams and
// double-buffered parameter snapshots, and the orchestration of Algorithm 1's learner,
// optimiser and gossip steps out of the kernels in the other sources.
#include <chrono>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <thread>

#include "internal.h"

using namespace gala;

constexpr long kFramePix = 84L * 84 * 4;

namespace {

struct Plan {  // one tensor-core product with its descriptors
    GemmOperand A, B;
    GemmArgs args;
    int tag = 0;
};
struct WgradPlan {  // conv2 / conv3 weight gradient with resident operands
    CUtensorMap x, y;
    WgradArgs args;
    int tag = 0;
};
struct Wgrad1Plan {  // conv1 weight gradient from the uint8 frames
    CUtensorMap y;
    Wgrad1Args args;
};
struct ConvPlan {  // one forward or data-gradient convolution (input resident in shared memory)
    CUtensorMap x, w;
    ConvArgs args;
    int tag = 0;
    bool built = false;
};

// Kernel classes for launch counting and optional per-class device timing.
enum Tag : int {
    T_CAST_FRAMES = 0, T_HEADS_FWD, T_LOSS, T_HEADS_BWD, T_COLSUM, T_SPLITK, T_GRAD_NORM,
    T_SWEEP_SYNC, T_SWEEP_AGENT, T_DENSE_FWD, T_DENSE_BWD, T_SAMPLE, T_CAST, T_HEADS_FUSED, T_ENV, T_MLP_FUSED,
    T_GEMM_CONV_FWD,          // +layer (3)
    T_GEMM_FC_FWD = T_GEMM_CONV_FWD + 3, T_GEMM_FC_WGRAD, T_GEMM_FC_DGRAD,
    T_GEMM_CONV_WGRAD,        // +layer (3)
    T_GEMM_CONV_DGRAD = T_GEMM_CONV_WGRAD + 3,  // +layer (3)
    T_COUNT = T_GEMM_CONV_DGRAD + 3
};
const char* const kTagNames[T_COUNT] = {
    "cast_frames", "heads_fwd", "a2c_loss", "heads_bwd", "colsum", "splitk_reduce", "grad_norm",
    "sweep_sync", "sweep_agent", "dense_fwd", "dense_bwd", "sample", "cast_bf16", "heads_fused", "env", "mlp_fused",
    "gemm_conv1_fwd", "gemm_conv2_fwd", "gemm_conv3_fwd", "gemm_fc_fwd", "gemm_fc_wgrad", "gemm_fc_dgrad",
    "gemm_conv1_wgrad", "gemm_conv2_wgrad", "gemm_conv3_wgrad", "gemm_conv1_dgrad", "gemm_conv2_dgrad",
    "gemm_conv3_dgrad"};

struct TimedLaunch { int tag; cudaEvent_t beg, end; };

// The kernels of one learner step (forward, objective, backward, norm) for a given set of rollout buffers,
// captured once as a CUDA graph: replaying it costs one launch on the host instead of ~17.
struct StepGraph {
    std::vector<const void*> key;   // streams, first agent, count, SM budget, the rollouts' pointers
    cudaGraphExec_t exec = nullptr;
    bool failed = false;            // capture or instantiation did not work: launch directly
    long long launches = 0;         // kernels inside
    long long tag_launches[T_COUNT] = {};
};

// Snapshot slots per agent: version w lives in slot w % kSnapSlots.  A reader takes one of the two newest versions,
// so with three slots the version that is written next never shares a slot with one that a sweep enqueued at the
// same time may read: agents that are each other's in-peers can publish and average in ONE launch.
constexpr int kSnapSlots = 3;

struct Agent {
    cudaStream_t stream = nullptr, lib_stream = nullptr;
    cudaEvent_t pub_event[kSnapSlots] = {};         // completion of the sweep that wrote snapshot slot s
    cudaEvent_t fence = nullptr;                    // scratch event for cross-stream ordering
    cudaStream_t sweep_stream = nullptr;            // stream the agent's latest sweep was enqueued on
    cudaStream_t pub_stream[kSnapSlots] = {};       // ... and the sweep that wrote slot s
    bool dirty = false;                             // its own stream carries work no group launch is ordered behind yet
    int group_lane = -1;                            // group lane whose work its own stream is not ordered behind yet
    long long version = 0;                          // newest snapshot version enqueued (0: none)
    long long round = 0;                            // local iteration counter
    bool pending = false;                           // a gradient waits for its optimiser step
    long long since_mix = 0;                        // local iterations since the last average with the in-peers
    std::vector<long long> consumed;                // newest version consumed from each agent
    std::vector<int> slot_readers[kSnapSlots];      // agents whose sweeps read snapshot slot s
    long long frames = 0, mixes = 0, skipped = 0, stale_sum = 0, stale_max = 0, stale_waits = 0;
    // closed actor loop: rollout buffers owned by the library and the environment's step counter
    void* loop_obs = nullptr; int* loop_actions = nullptr; float* loop_rewards = nullptr;
    unsigned char* loop_dones = nullptr; float* loop_uniforms = nullptr;
    long long* env_step_dev = nullptr;              // the step counter the environment kernels read
    long long env_step = 0;                         // its host mirror (steps enqueued so far)
    StepGraph loop_graph;                           // one loop iteration (act, environment, learn) as a graph
    unsigned long long loop_seed = 0; int loop_seen = 0;
    int last_n = 0, last_mixed = 0;
    int last_peers[2] = {0, 0};
    long long last_versions[2] = {0, 0};
};

}  // namespace

struct gala_ctx {
    int n = 0;
    gala_topology topo{};
    gala_net_spec net{};
    gala_hparams hp{};
    long d = 0, d_pad = 0;
    int T = 0, E = 0, A = 0, H = 0, obs_dim = 0;
    long B = 0, S = 0;
    bool conv = false;
    ConvLayout cl{};
    MlpLayout ml{};
    std::vector<Agent> agents;
    cudaStream_t main_stream = nullptr;
    cudaEvent_t main_event = nullptr;
    // second stream of the synchronous mode: the weight gradients of heads, hidden layer, conv3 and conv2 run beside the chain
    // of data gradients they do not depend on
    cudaStream_t side_stream = nullptr;
    // third stream of the synchronous mode: the column sums (bias gradients) run beside conv1's weight gradient, both
    // behind the last data gradient
    cudaStream_t tail_stream = nullptr;
    cudaEvent_t ev_tail_fork = nullptr, ev_tail_join = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // Streams of the grouped per-agent calls (gala_learn_many / gala_gossip_many): a launch set for a list of agents
    // goes to one lane (its stream, a side stream for the weight gradients); consecutive calls alternate between the
    // lanes so that the tail of one set overlaps the head of the next.
    struct Lane { cudaStream_t st = nullptr, side = nullptr; cudaEvent_t fork = nullptr, join = nullptr, done = nullptr; };
    Lane glane[2];
    int n_lanes = 1, next_lane = 0;
    const AgentMap* cur_map = nullptr;       // agent list of the launches being enqueued (null: a range of agents)
    cudaEvent_t cur_fork = nullptr, cur_join = nullptr;   // fork / join events of the stream pair in use
    // closed actor loops: rollout buffers of all agents, one block per kind (an agent's loop_* pointers are slices)
    uint8_t* la_obs = nullptr; int* la_actions = nullptr; float* la_rewards = nullptr; unsigned char* la_dones = nullptr;
    float* la_uniforms = nullptr; long long* la_steps = nullptr;
    StepGraph la_graph;                      // the acting part of one lockstep iteration (all agents) as a graph
    unsigned long long la_seed = 0; int la_seen = 0;
    long long sync_round = 0;
    long long launches = 0;
    long long tag_launches[T_COUNT] = {};
    unsigned long long profile_mask = 0;     // kernel classes bracketed by timing events
    std::vector<TimedLaunch> timed;          // recorded, not yet read
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> event_pool;
    std::string err;
    std::vector<void*> allocs;

    float *x = nullptr, *g = nullptr, *v = nullptr, *snap = nullptr;
    __nv_bfloat16* shadow = nullptr;
    float *clip = nullptr, *norm = nullptr, *losses = nullptr;
    double *norm_partial = nullptr, *colsum_partial = nullptr;
    unsigned *norm_ticket = nullptr, *colsum_ticket = nullptr, *heads_ticket = nullptr;
    float* c1b = nullptr;                    // bias-gradient slices of conv1, left by conv2's data gradient
    long c1b_min_samples = 2048;             // ... in launches over at least this many samples
    int fc_bn = 128;                         // columns of a tile of the hidden layer's forward product
    float* fc_sq = nullptr;                  // [N][1600] sums of squares of the hidden layer's weight gradient, by 32 x 32 block
    float* dzv = nullptr;                    // [N][S][20] rows (dlogits, dvalue, zeros) of the fused heads kernel
    float* heads_partial = nullptr;          // [N][E][4] objective sums per block of the fused heads kernel
    bool fused_heads = false;
    bool fused_mlp = false;                  // the MLP learner step as one kernel
    float* mlp_partial = nullptr;            // [N][kMlpMaxBlocks][d + 4] partial gradients of its blocks
    int use_graphs = 1;                      // replay a learner step whose rollout buffers were seen before as a graph:
                                             // 0 never, 1 in the synchronous round, 2 also in the per-agent calls
    std::vector<StepGraph> graphs;
    int agent_ctas = 0;                      // SM budget of one agent's kernels in the per-agent calls (0: all)
    ReduceSegs pending{};                    // sliced conv weight gradients of the step that still wait for their sum
    long splitk_region[3] = {0, 0, 0};       // offset of conv layer l's slices inside an agent's split-K workspace
    long bias_region[3] = {0, 0, 0};         // ... and of the slices of its bias gradient (64 floats each; conv2, conv3)
    int cur_ctas = 0;                        // budget of the launches being enqueued (0 in the synchronous round)
    int* error_word = nullptr;
    double *cons_partial = nullptr, *cons_out = nullptr;
    unsigned* cons_ticket = nullptr;
    // update-norm tracking (Proposition 1): ||alpha G||_F^2 of the last synchronous round
    bool track_updates = false;
    bool upd_valid = false;
    double *upd_partial = nullptr, *upd_out = nullptr;
    unsigned* upd_ticket = nullptr;
    int stale_timeout_ms = 1000;   // longest host wait of a staleness-bounded gossip step
    float *logits = nullptr, *values = nullptr, *returns = nullptr, *adv = nullptr, *dlogits = nullptr,
          *dvalues = nullptr;
    // MLP workspaces
    float *h1 = nullptr, *h2 = nullptr, *dpre1 = nullptr, *dpre2 = nullptr;
    // conv workspaces (bf16)
    __nv_bfloat16* frames = nullptr;   // bf16 copies of the uint8 frames, [N][B][84][84][4]
    __nv_bfloat16* act[3] = {nullptr, nullptr, nullptr};
    __nv_bfloat16 *hid = nullptr, *dh = nullptr, *dy[3] = {nullptr, nullptr, nullptr};
    float* splitk_ws = nullptr;
    long splitk_group_stride = 0;
    int max_split = 32;
    Plan fwd[3], fc_fwd, fc_wgrad, fc_dgrad, wgrad[3], dgrad[3];
    ConvPlan cfwd[3], cdgrad[3];
    WgradPlan cwgrad[3];
    Wgrad1Plan cwgrad1;
    uint32_t* gate[3] = {nullptr, nullptr, nullptr};   // ReLU gate bits of act[0..2]
    bool legacy_conv = false;
};

namespace {

int fail(gala_ctx* c, int code, const char* fmt, ...) {
    if (c) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        c->err = buf;
    }
    return code;
}
#define CK(call)                                                                                       \
    do {                                                                                               \
        cudaError_t e__ = (call);                                                                      \
        if (e__ != cudaSuccess)                                                                        \
            return fail(c, e__ == cudaErrorMemoryAllocation ? GALA_ENOMEM : GALA_ECUDA, "%s: %s", #call, \
                        cudaGetErrorString(e__));                                                      \
    } while (0)
// Launch bookkeeping: counts every kernel launch per class; classes selected by profile_mask are
// bracketed by timing events on the launching stream.
int prof_begin(gala_ctx* c, int tag, cudaStream_t st, TimedLaunch* t) {
    t->tag = -1;
    if (!((c->profile_mask >> tag) & 1ull)) return GALA_OK;
    if (c->event_pool.empty()) {
        cudaEvent_t a, b;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess)
            return fail(c, GALA_ECUDA, "cudaEventCreate failed");
        c->event_pool.push_back({a, b});
    }
    t->beg = c->event_pool.back().first; t->end = c->event_pool.back().second;
    c->event_pool.pop_back();
    t->tag = tag;
    if (cudaEventRecord(t->beg, st) != cudaSuccess) return fail(c, GALA_ECUDA, "cudaEventRecord failed");
    return GALA_OK;
}
int prof_end(gala_ctx* c, cudaStream_t st, TimedLaunch* t) {
    if (t->tag < 0) return GALA_OK;
    if (cudaEventRecord(t->end, st) != cudaSuccess) return fail(c, GALA_ECUDA, "cudaEventRecord failed");
    c->timed.push_back(*t);
    return GALA_OK;
}
#define LAUNCH(tag, st, call)                                    \
    do {                                                         \
        TimedLaunch tl__;                                        \
        int pr__ = prof_begin(c, (tag), (st), &tl__);            \
        if (pr__ != GALA_OK) return pr__;                        \
        CK(call);                                                \
        c->launches++;                                           \
        c->tag_launches[(tag)]++;                                \
        if ((pr__ = prof_end(c, (st), &tl__)) != GALA_OK) return pr__; \
    } while (0)

template <typename Tp>
int dev_alloc(gala_ctx* c, Tp** p, size_t count) {
    void* q = nullptr;
    size_t bytes = count * sizeof(Tp);
    if (bytes == 0) bytes = 16;
    cudaError_t e = cudaMalloc(&q, bytes);
    if (e != cudaSuccess) return fail(c, GALA_ENOMEM, "cudaMalloc(%zu bytes): %s", bytes, cudaGetErrorString(e));
    e = cudaMemset(q, 0, bytes);
    if (e != cudaSuccess) return fail(c, GALA_ECUDA, "cudaMemset: %s", cudaGetErrorString(e));
    c->allocs.push_back(q);
    *p = reinterpret_cast<Tp*>(q);
    return GALA_OK;
}
#define ALLOC(ptr, count)                       \
    do {                                        \
        int r__ = dev_alloc(c, &(ptr), (count)); \
        if (r__ != GALA_OK) return r__;         \
    } while (0)

// ------------------------------------------------------------------ topology (integers only)
// In-peers of `agent` at round `round`.
//   ring: directed ring v_0 -> v_1 -> ... -> v_0, in-peers i-1 .. i-p (Appendix C.2, Fig. 5)
//   exponential: L = ceil(log2 n); j-th in-peer is i - 2^((p*round + j) mod L)
// Coinciding peers are kept as separate terms so the weights stay 1/(1+p).
int topo_offsets(const gala_topology& t, int n, long long round, int* off) {
    if (n <= 1) return 0;
    if (t.kind == GALA_TOPO_RING) {
        for (int j = 0; j < t.peers; j++) off[j] = (j + 1) % n;
        return t.peers;
    }
    int L = 0;
    while ((1LL << L) < n) L++;
    if (L < 1) L = 1;
    for (int j = 0; j < t.peers; j++) {
        long long e = ((long long)t.peers * round + j) % L;
        off[j] = (int)((1LL << e) % n);
    }
    return t.peers;
}

// ------------------------------------------------------------------ initial parameters
// Counter-based generator: SplitMix64 finaliser applied to (seed, agent, index).
inline uint64_t splitmix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
inline float uniform_pm1(uint64_t seed, uint64_t agent, uint64_t idx) {
    uint64_t h = splitmix64(splitmix64(seed ^ (agent * 0xD1342543DE82EF95ull)) + idx);
    return (float)((double)(h >> 11) * (1.0 / 9007199254740992.0) * 2.0 - 1.0);
}
void init_tensor(float* p, long off, long count, int fan_in, uint64_t seed, uint64_t agent) {
    const float s = 1.0f / std::sqrt((float)fan_in);
    for (long i = 0; i < count; i++) p[off + i] = s * uniform_pm1(seed, agent, (uint64_t)(off + i));
}

void fill_batch(PtrBatch& pb, const void* base, long stride_bytes, int agent0, int count) {
    for (int i = 0; i < count; i++) pb.p[i] = reinterpret_cast<const char*>(base) + (long)(agent0 + i) * stride_bytes;
}

// Agents of the launches being enqueued: k-th agent of a launch over [agent0, agent0 + groups), or of the list in use
// (then agent0 is 0 and every base pointer is agent 0's).
inline int sel_agent(const gala_ctx* c, int agent0, int k) { return c->cur_map ? (int)c->cur_map->v[k] : agent0 + k; }
inline AgentMap sel_map(const gala_ctx* c) { return c->cur_map ? *c->cur_map : AgentMap{}; }

// ------------------------------------------------------------------ GEMM plans (conv net)
int build_plans(gala_ctx* c) {
    const int n = c->n;
    const long B = c->B, S = c->S, dp = c->d_pad;
    const int P[3] = {400, 81, 49};
    auto zero_args = [&](Plan& p) {
        memset(&p.args, 0, sizeof p.args);
        p.args.groups = n; p.args.split_k = 1; p.args.scale = 1.0f; p.args.error_word = c->error_word;
    };
    bool ok = true;
    for (int l = 0; l < 3; l++) {
        const int KK = kConvKK[l], CO = kConvCout[l];
        const int bn = CO;  // 32 or 64
        // forward: patches [B*P][KK] x W[CO][KK]^T -> act[l] (bias, ReLU; conv1 also 1/255)
        Plan& f = c->fwd[l];
        zero_args(f);
        f.tag = T_GEMM_CONV_FWD + l;
        // conv2 / conv3 read their patches straight from the previous layer's activations: one TMA box
        // per kernel offset holds the [patch][channel] block of nb samples (see gemm.cu, CONV_FWD)
        const int nb = l == 1 ? 1 : 2;
        if (l == 0) {
            // bf16 frames [sample][84][84][4] seen as [sample][y/4][y%4][ox][8 px x 4 ch]: the 20 windows of a
            // row overlap by half (stride 4 px = 32 B under a 64 B extent); one box = one kernel row of the
            // 100 patches of a quarter sample
            const uint64_t dims[5] = {32, 20, 4, 21, (uint64_t)n * B};
            const uint64_t str[4] = {32, 672, 2688, 56448};
            const uint32_t box[5] = {32, 20, 1, 5, 1};
            ok &= make_tensor_map_nd(&f.A.map, c->frames, 5, dims, str, box, 1);
            f.A.mn_major = 0;
        } else if (l == 1) {   // act1 [sample][20][20][32] seen as [sample][y/2][y%2][x/2][2 px x 32 ch]
            const uint64_t dims[5] = {64, 10, 2, 10, (uint64_t)n * B};
            const uint64_t str[4] = {128, 1280, 2560, 25600};
            const uint32_t box[5] = {64, 9, 1, 9, 1};
            ok &= make_tensor_map_nd(&f.A.map, c->act[0], 5, dims, str, box);
            f.A.mn_major = 0;
        } else {               // act2 [sample][9][9][64]
            const uint64_t dims[4] = {64, 9, 9, (uint64_t)n * B};
            const uint64_t str[3] = {128, 1152, 10368};
            const uint32_t box[4] = {64, 7, 7, (uint32_t)nb};
            ok &= make_tensor_map_nd(&f.A.map, c->act[1], 4, dims, str, box);
            f.A.mn_major = 0;
        }
        f.args.conv_mode = CONV_FWD; f.args.conv_layer = l; f.args.conv_nb = nb; f.args.a_samples = (int)B;
        if (l == 0) {
            f.args.conv_nb = 1; f.args.tile_rows = 100; f.args.box_rows = 100;
            f.args.kpack = 4; f.args.k_steps = 8 / f.args.kpack;   // 4 kernel rows per K step
            const uint64_t wd[3] = {(uint64_t)KK, (uint64_t)CO, (uint64_t)n};
            const uint64_t ws[2] = {(uint64_t)KK * 2, (uint64_t)dp * 2};
            const uint32_t wb[3] = {32, 32, 1};
            ok &= make_tensor_map_nd(&f.B.map, c->shadow + c->cl.w[0], 3, wd, ws, wb, 1);
            f.B.mn_major = 0;
        } else {
            f.args.tile_rows = nb * P[l]; f.args.box_rows = nb * P[l]; f.args.k_steps = KK / 64;
            f.args.kpack = 2;   // two kernel offsets per K step
            ok &= make_operand(&f.B, c->shadow + c->cl.w[l], 0, CO, KK, n, KK, dp, bn);
        }
        f.args.M = (int)(B * P[l]); f.args.N = CO; f.args.K = KK; f.args.block_n = bn;
        f.args.flags = EPI_OUT_BF16 | EPI_RELU;
        f.args.scale = l == 0 ? 1.0f / 255.0f : 1.0f;
        f.args.bias = c->x + c->cl.b[l]; f.args.bias_group_stride = dp;
        f.args.out = c->act[l]; f.args.out_group_stride = B * P[l] * CO; f.args.ldc = CO;
        // weight gradient, transposed product: (patches^T [KK x S*P]) x (dY [S*P x CO]) stored at W[co][kk]
        Plan& w = c->wgrad[l];
        zero_args(w);
        w.tag = T_GEMM_CONV_WGRAD + l;
        if (l == 0) {
            // transposed patch matrix from the same frame boxes (4 kernel rows = 128 patch elements per M
            // tile); dY1 [sample][400][32] in boxes of the 100 patches of a quarter sample
            w.A = f.A; w.A.mn_major = 1;
            const uint64_t dims[3] = {32, 400, (uint64_t)n * S};
            const uint64_t str[2] = {64, 25600};
            const uint32_t box[3] = {32, 100, 1};
            ok &= make_tensor_map_nd(&w.B.map, c->dy[0], 3, dims, str, box, 1);
            w.B.mn_major = 1;
            w.args.conv_mode = CONV_WGRAD; w.args.conv_layer = 0; w.args.conv_nb = 1;
            w.args.a_samples = (int)B; w.args.b_samples = (int)S;
            w.args.kstep_rows = 112; w.args.tile_rows = 128; w.args.box_rows = 100; w.args.k_steps = (int)(S * 4);
        } else {
            // same activation boxes as the forward pass, now as the transposed patch matrix; dY comes in
            // boxes of whole samples too, so that one K step is the patches of nb samples
            w.A = f.A; w.A.mn_major = 1;
            const uint64_t dims[4] = {64, (uint64_t)P[l], (uint64_t)S, (uint64_t)n};
            const uint64_t str[3] = {128, (uint64_t)P[l] * 128, (uint64_t)S * P[l] * 128};
            const uint32_t box[4] = {64, (uint32_t)P[l], (uint32_t)nb, 1};
            ok &= make_tensor_map_nd(&w.B.map, c->dy[l], 4, dims, str, box);
            w.B.mn_major = 1;
            w.args.conv_mode = CONV_WGRAD; w.args.conv_layer = l; w.args.conv_nb = nb;
            w.args.a_samples = (int)B; w.args.b_samples = (int)S;
            w.args.kstep_rows = l == 1 ? 96 : 112;
            w.args.tile_rows = 128; w.args.box_rows = nb * P[l]; w.args.k_steps = (int)((S + nb - 1) / nb);
        }
        w.args.M = KK; w.args.N = CO; w.args.K = (int)(S * P[l]); w.args.block_n = l == 0 ? 32 : 64;
        w.args.flags = EPI_TRANSPOSE;
        w.args.scale = l == 0 ? 1.0f / 255.0f : 1.0f;
        w.args.out = c->g + c->cl.w[l]; w.args.out_group_stride = dp; w.args.ldc = KK;
        // data gradient (conv2, conv3), implicit: the gradient of the layer's INPUT pixels is summed over the
        // kernel offsets inside the accumulator (no patch gradients in memory), gated by the ReLU of the
        // input activation in the epilogue and stored as the previous layer's dY
        if (l > 0) {
            Plan& dg = c->dgrad[l];
            zero_args(dg);
            dg.tag = T_GEMM_CONV_DGRAD + l;
            const int ow = kConvOut[l], in_pix = kConvIn[l] * kConvIn[l], cin = kConvCin[l];
            const uint64_t dims[4] = {64, (uint64_t)ow, (uint64_t)ow, (uint64_t)n * S};
            const uint64_t str[3] = {128, (uint64_t)ow * 128, (uint64_t)ow * ow * 128};
            const uint32_t box[4] = {64, l == 2 ? 9u : 10u, l == 2 ? 9u : 10u, 1};
            ok &= make_tensor_map_nd(&dg.A.map, c->dy[l], 4, dims, str, box);
            dg.A.mn_major = 0;
            const uint64_t wd[3] = {(uint64_t)KK, (uint64_t)CO, (uint64_t)n};
            const uint64_t ws[2] = {(uint64_t)KK * 2, (uint64_t)dp * 2};
            const uint32_t wb[3] = {64, 64, 1};
            ok &= make_tensor_map_nd(&dg.B.map, c->shadow + c->cl.w[l], 3, wd, ws, wb);
            dg.B.mn_major = 1;
            dg.args.M = (int)(S * in_pix); dg.args.N = cin; dg.args.K = KK; dg.args.block_n = 64;
            dg.args.conv_mode = CONV_DGRAD; dg.args.conv_layer = l; dg.args.conv_nb = 1; dg.args.a_samples = (int)S;
            dg.args.tile_rows = l == 2 ? 81 : 100; dg.args.box_rows = dg.args.tile_rows;
            dg.args.k_steps = l == 2 ? 9 : 4;
            dg.args.kpack = 2;  // two kernel offsets per K step
            dg.args.flags = EPI_OUT_BF16 | EPI_MASK | (l == 1 ? EPI_ROWMAP_S2 : 0);
            dg.args.mask = c->act[l - 1]; dg.args.mask_group_stride = B * in_pix * cin;
            dg.args.out = c->dy[l - 1]; dg.args.out_group_stride = S * in_pix * cin; dg.args.ldc = cin;
        }
    }
    {   // hidden layer forward: act3 [B][3136] x Wfc[512][3136]^T -> hid (bias, ReLU)
        Plan& f = c->fc_fwd;
        zero_args(f);
        f.tag = T_GEMM_FC_FWD;
        // forward: 128 x 256 tiles (one CTA an SM; a quarter less operand traffic from L2, which bounds this product
        // with its 3136-long reduction) once an agent's batch fills several row tiles; 128 x 128 below that, where
        // the number of CTAs matters more
        const int fbn = c->fc_bn;
        ok &= make_operand(&f.A, c->act[2], 0, B, kFeat, n, kFeat, (uint64_t)B * kFeat, 128);
        ok &= make_operand(&f.B, c->shadow + c->cl.fcw, 0, kHidden, kFeat, n, kFeat, dp, fbn);
        f.args.M = (int)B; f.args.N = kHidden; f.args.K = kFeat; f.args.block_n = fbn;
        f.args.flags = EPI_OUT_BF16 | EPI_RELU;
        f.args.bias = c->x + c->cl.fcb; f.args.bias_group_stride = dp;
        f.args.out = c->hid; f.args.out_group_stride = B * kHidden; f.args.ldc = kHidden;
        // weight gradient: dh^T [512 x S] x act3 [S x 3136] -> gW[512][3136]
        Plan& w = c->fc_wgrad;
        zero_args(w);
        w.tag = T_GEMM_FC_WGRAD;
        ok &= make_operand(&w.A, c->dh, 1, kHidden, S, n, kHidden, (uint64_t)S * kHidden, 128);
        ok &= make_operand(&w.B, c->act[2], 1, kFeat, S, n, kFeat, (uint64_t)B * kFeat, 128);
        w.args.M = kHidden; w.args.N = kFeat; w.args.K = (int)S; w.args.block_n = 128;   // (bound by its epilogue: no gain from wider tiles)
        w.args.out = c->g + c->cl.fcw; w.args.out_group_stride = dp; w.args.ldc = kFeat;
        w.args.sq_partial = c->fc_sq;   // so that the norm pass need not read these 95 % of the gradient again
        // data gradient: dh [S][512] x Wfc [512][3136] -> dY3 [S][3136], masked by act3 > 0
        Plan& dg = c->fc_dgrad;
        zero_args(dg);
        dg.tag = T_GEMM_FC_DGRAD;
        ok &= make_operand(&dg.A, c->dh, 0, S, kHidden, n, kHidden, (uint64_t)S * kHidden, 128);
        ok &= make_operand(&dg.B, c->shadow + c->cl.fcw, 1, kFeat, kHidden, n, kFeat, dp, 128);
        dg.args.M = (int)S; dg.args.N = kFeat; dg.args.K = kHidden; dg.args.block_n = 128;
        if (c->legacy_conv) {   // the legacy conv3 forward writes no gate bits: gate on the stored activation itself
            dg.args.flags = EPI_OUT_BF16 | EPI_MASK;
            dg.args.mask = c->act[2]; dg.args.mask_group_stride = B * kFeat;
        } else {                // one gate word per row and 32 columns instead of 64 bytes of activations
            dg.args.flags = EPI_OUT_BF16 | EPI_GATE;
            dg.args.gate = c->gate[2]; dg.args.gate_group_stride = B * kFeat / 32;
        }
        dg.args.out = c->dy[2]; dg.args.out_group_stride = S * kFeat; dg.args.ldc = kFeat;
    }
    for (int l = 0; l < 3; l++) {
        const int CO = kConvCout[l];
        ConvPlan& f = c->cfwd[l];
        memset(&f.args, 0, sizeof f.args);
        f.tag = T_GEMM_CONV_FWD + l;
        f.args.variant = CV_CONV1_FWD + l;
        f.args.a_samples = (int)B;
        // conv1's products take the weights as fp16(w * 2^12) and the frames as the integers they are
        f.args.scale = l == 0 ? 1.0f / (255.0f * 4096.0f) : 1.0f;
        f.args.bias = c->x + c->cl.b[l]; f.args.bias_group_stride = dp;
        f.args.out = c->act[l]; f.args.out_group_stride = B * P[l] * CO;
        f.args.gate_out = c->gate[l]; f.args.gate_group_stride = B * P[l] * CO / 32;
        f.args.error_word = c->error_word;
        const void* xin = l == 0 ? (const void*)c->frames : (const void*)c->act[l - 1];
        ok &= make_conv_maps(f.args.variant, &f.x, &f.w, xin, (uint64_t)n * B, c->shadow + c->cl.w[l], n, dp);
        f.built = true;
        if (l > 0) {
            WgradPlan& wg = c->cwgrad[l];
            memset(&wg.args, 0, sizeof wg.args);
            wg.tag = T_GEMM_CONV_WGRAD + l;
            wg.args.variant = l == 1 ? WG_CONV2 : WG_CONV3;
            wg.args.x_samples = (int)B; wg.args.y_samples = (int)S; wg.args.samples = (int)S;
            wg.args.out = c->g + c->cl.w[l]; wg.args.out_group_stride = dp;
            wg.args.error_word = c->error_word;
            ok &= make_wgrad_maps(wg.args.variant, &wg.x, &wg.y, c->act[l - 1], (uint64_t)n * B, c->dy[l], (uint64_t)n * S);
            ConvPlan& d = c->cdgrad[l];
            memset(&d.args, 0, sizeof d.args);
            d.tag = T_GEMM_CONV_DGRAD + l;
            d.args.variant = l == 1 ? CV_CONV2_DGRAD : CV_CONV3_DGRAD;
            d.args.a_samples = (int)S;
            d.args.scale = 1.0f;
            const long in_elems = (long)kConvIn[l] * kConvIn[l] * kConvCin[l];
            d.args.gate_in = c->gate[l - 1]; d.args.gate_group_stride = B * in_elems / 32;
            d.args.out = c->dy[l - 1]; d.args.out_group_stride = S * in_elems;
            d.args.error_word = c->error_word;
            if (l == 1) d.args.bias_partial = c->c1b;   // per-channel sums of dY1 = conv1's bias gradient
            ok &= make_conv_maps(d.args.variant, &d.x, &d.w, c->dy[l], (uint64_t)n * S, c->shadow + c->cl.w[l], n, dp);
            d.built = true;
        }
    }
    {
        Wgrad1Plan& w1 = c->cwgrad1;
        memset(&w1.args, 0, sizeof w1.args);
        w1.args.samples = (int)S; w1.args.y_samples = (int)S;
        w1.args.scale = 1.0f / 255.0f;
        w1.args.out = c->g + c->cl.w[0]; w1.args.out_group_stride = dp;
        w1.args.error_word = c->error_word;
        ok &= make_wgrad1_map(&w1.y, c->dy[0], (uint64_t)n * S);
    }
    return ok ? GALA_OK : fail(c, GALA_ECUDA, "cuTensorMapEncodeTiled failed while building GEMM descriptors");
}


// Slices of the samples per agent for a weight gradient whose CTAs each own one agent and a slice: chosen so
// that the CTAs fill the SMs in whole waves.  `fixed` = set-up and epilogue of a CTA in units of one sample.
int pick_splits(gala_ctx* c, int groups, int S, long count, int fixed) {
    int best = 1;
    long best_cost = -1;
    const long sms = c->cur_ctas > 0 ? c->cur_ctas : sm_count();
    for (int sp = 1; sp <= c->max_split && sp <= S; sp++) {
        if (sp > 1 && S / sp < 4) break;   // max_split slices of every layer fit its region of the workspace
        if (sp > 1 && c->cur_ctas > 0 && (long)groups * sp > sms) break;
        const long waves = ((long)groups * sp + sms - 1) / sms, per = (S + sp - 1) / sp;
        const long cost = waves * (per + fixed) + (sp > 1 ? 8 : 0);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = sp; }
    }
    return best;
}

// conv1 weight gradient from the uint8 frames; with more than one slice the partial sums go through the
// fixed-order reduction
int run_conv1_wgrad(gala_ctx* c, int agent0, int groups, const PtrBatch& obs, cudaStream_t st) {
    Wgrad1Args a = c->cwgrad1.args;
    const long count = 32 * 256;
    a.group0 = agent0; a.groups = groups; a.obs = obs; a.am = sel_map(c);
    a.splits = pick_splits(c, groups, a.samples, count, 3);
    float* final_out = a.out + (long)agent0 * a.out_group_stride;
    if (a.splits == 1) {
        a.out = final_out; a.out_split_stride = 0;
        LAUNCH(T_GEMM_CONV_WGRAD, st, launch_wgrad1(c->cwgrad1.y, a, st));
        return GALA_OK;
    }
    float* ws = c->splitk_ws + (long)agent0 * c->splitk_group_stride;
    a.out = ws + c->splitk_region[0];
    a.out_group_stride = c->splitk_group_stride; a.out_split_stride = count;
    // (conv1's bias gradient stays with the column-sum kernel: all warps of this kernel are busy converting, and one
    // more warp that summed the dY tiles became its bottleneck, 0.19 -> 0.37 ms at 16 agents x 640 samples)
    LAUNCH(T_GEMM_CONV_WGRAD, st, launch_wgrad1(c->cwgrad1.y, a, st));
    c->pending.s[c->pending.n++] = ReduceSeg{c->cl.w[0], count, c->splitk_region[0], a.splits};
    return GALA_OK;
}

// conv2 / conv3 weight gradient: slices of the samples per agent chosen so that the CTAs fill the SMs in
// whole waves; with more than one slice the partial sums go through the fixed-order reduction
int run_conv_wgrad(gala_ctx* c, const WgradPlan& p, int agent0, int groups, cudaStream_t st) {
    WgradArgs a = p.args;
    const int S = a.samples;
    const long count = (long)(a.variant == WG_CONV2 ? 64 * 512 : 64 * 576);
    const int best = pick_splits(c, groups, S, count, 6);
    a.group0 = agent0; a.groups = groups; a.splits = best; a.am = sel_map(c);
    const int l = a.variant == WG_CONV2 ? 1 : 2;
    if (best == 1) {
        a.out += (long)agent0 * a.out_group_stride;
        a.out_split_stride = 0;
        a.bias_out = c->g + (long)agent0 * c->d_pad + c->cl.b[l]; a.bias_group_stride = c->d_pad; a.bias_split_stride = 0;
        LAUNCH(p.tag, st, launch_wgrad(p.x, p.y, a, st));
        return GALA_OK;
    }
    float* ws = c->splitk_ws + (long)agent0 * c->splitk_group_stride;
    a.out = ws + c->splitk_region[l];
    a.out_group_stride = c->splitk_group_stride; a.out_split_stride = count;
    a.bias_out = ws + c->bias_region[l]; a.bias_group_stride = c->splitk_group_stride; a.bias_split_stride = 64;
    LAUNCH(p.tag, st, launch_wgrad(p.x, p.y, a, st));
    c->pending.s[c->pending.n++] = ReduceSeg{c->cl.w[l], count, c->splitk_region[l], best};
    c->pending.s[c->pending.n++] = ReduceSeg{c->cl.b[l], 64, c->bias_region[l], best};
    return GALA_OK;
}

// One launch adds up the slices of every conv weight gradient that was sliced in this step.
int flush_pending_reduces(gala_ctx* c, int agent0, int groups, cudaStream_t st) {
    if (c->pending.n == 0) return GALA_OK;
    const ReduceSegs segs = c->pending;
    c->pending.n = 0;
    LAUNCH(T_SPLITK, st, launch_splitk_reduce_multi(c->splitk_ws + (long)agent0 * c->splitk_group_stride,
                                                   c->g + (long)agent0 * c->d_pad, segs, groups, c->splitk_group_stride,
                                                   c->d_pad, st, c->cur_map));
    return GALA_OK;
}

int run_conv(gala_ctx* c, const ConvPlan& p, int agent0, int groups, int rows, cudaStream_t st,
             const PtrBatch* obs = nullptr) {
    ConvArgs a = p.args;
    if (obs) a.obs = *obs;
    a.group0 = agent0; a.groups = groups; a.rows = rows; a.max_ctas = c->cur_ctas; a.am = sel_map(c);
    a.out += (long)agent0 * a.out_group_stride;
    if (a.gate_out) a.gate_out += (long)agent0 * a.gate_group_stride;
    if (a.gate_in) a.gate_in += (long)agent0 * a.gate_group_stride;
    if (a.bias_partial) {
        if ((long)groups * rows < c->c1b_min_samples) a.bias_partial = nullptr;
        else a.bias_partial += (long)agent0 * kConvBiasSliceStride;
    }
    LAUNCH(p.tag, st, launch_conv(p.x, p.w, a, st));
    return GALA_OK;
}

int run_plan(gala_ctx* c, const Plan& p, int agent0, int groups, int m_override, cudaStream_t st) {
    GemmArgs a = p.args;
    a.group0 = agent0; a.groups = groups; a.max_ctas = c->cur_ctas; a.am = sel_map(c);
    if (m_override > 0) a.M = m_override;
    const bool bf = a.flags & EPI_OUT_BF16;
    a.out = reinterpret_cast<char*>(a.out) + (long)agent0 * a.out_group_stride * (bf ? 2 : 4);
    if (a.mask) a.mask += (long)agent0 * a.mask_group_stride;
    if (a.gate) a.gate += (long)agent0 * a.gate_group_stride;
    if (a.sq_partial) a.sq_partial += (long)agent0 * ((a.M + 127) / 128) * ((a.N + a.block_n - 1) / a.block_n) * (a.block_n / 8);
    LAUNCH(p.tag, st, launch_gemm(p.A, p.B, a, st));
    return GALA_OK;
}

// weight-gradient product with the reduction split over CTAs and a fixed-order second stage
int run_wgrad(gala_ctx* c, const Plan& p, int agent0, int groups, cudaStream_t st) {
    const int k_tiles = p.args.conv_mode != CONV_NONE ? p.args.k_steps : (p.args.K + 63) / 64;
    const int tiles = ((p.args.M + 127) / 128) * ((p.args.N + p.args.block_n - 1) / p.args.block_n);
    int split = (2 * sm_count()) / (groups * tiles);
    if (split > k_tiles / 4) split = k_tiles / 4;
    if (split > c->max_split) split = c->max_split;
    if (split < 1) split = 1;
    if (split == 1) return run_plan(c, p, agent0, groups, 0, st);
    GemmArgs a = p.args;
    const long count = (long)p.args.M * p.args.N;
    a.group0 = agent0; a.groups = groups; a.split_k = split; a.max_ctas = c->cur_ctas; a.am = sel_map(c);
    a.out = c->splitk_ws + (long)agent0 * c->splitk_group_stride;
    a.out_group_stride = c->splitk_group_stride;
    a.out_split_stride = count;
    LAUNCH(p.tag, st, launch_gemm(p.A, p.B, a, st));
    LAUNCH(T_SPLITK, st, launch_splitk_reduce(c->splitk_ws + (long)agent0 * c->splitk_group_stride,
                                reinterpret_cast<float*>(p.args.out) + (long)agent0 * p.args.out_group_stride, count,
                                split, count, groups, c->splitk_group_stride, p.args.out_group_stride, st));
    return GALA_OK;
}

// ------------------------------------------------------------------ forward / backward
// Forward on `rows` observations per agent for agents [agent0, agent0+groups).
// What forward() leaves undone when the caller fuses the heads with the objective: the hidden layer's
// split-K partial sums (split > 1) still wait for their reduction, bias and ReLU.
struct HiddenPending { int split = 0; long count = 0; };

// frames_st: stream on which the bf16 copies of the frames are made (they feed the legacy conv1 products);
// null: no copy.
// pend != null: stop before the heads (and before the reduction of a split hidden-layer product).
int forward(gala_ctx* c, int agent0, int groups, const PtrBatch& obs, int rows, cudaStream_t st,
            cudaStream_t frames_st, HiddenPending* pend = nullptr) {
    const long dp = c->d_pad, B = c->B;
    if (c->conv) {
        const int P[3] = {400, 81, 49};
        for (int i = 0; i < groups; i++)
            if (reinterpret_cast<uintptr_t>(obs.p[i]) & 15)
                return fail(c, GALA_EINVAL, "uint8 observations must be 16-byte aligned");
        if (frames_st)
            LAUNCH(T_CAST_FRAMES, frames_st, launch_cast_frames(obs, c->frames + (long)agent0 * B * kFramePix, B * kFramePix, rows, groups, frames_st));
        for (int l = 0; l < 3; l++) {
            int r = c->legacy_conv ? run_plan(c, c->fwd[l], agent0, groups, rows * P[l], st)
                                   : run_conv(c, c->cfwd[l], agent0, groups, rows, st, l == 0 ? &obs : nullptr);
            if (r != GALA_OK) return r;
        }
        // hidden layer: with few rows there are only a handful of output tiles, each streaming 0.8 MB of
        // weights through one SM; split the 3136-long reduction over more CTAs then
        int r;
        {
            const Plan& p = c->fc_fwd;
            const int tiles = ((rows + 127) / 128) * (kHidden / p.args.block_n);
            int split = (c->cur_ctas > 0 ? 2 * c->cur_ctas : 2 * sm_count()) / (groups * tiles);
            if (split > 7) split = 7;
            while (split > 1 && (long)split * rows * kHidden > c->splitk_group_stride) split--;
            if (split <= 1) {
                r = run_plan(c, p, agent0, groups, rows, st);
                if (r != GALA_OK) return r;
            } else {
                GemmArgs a = p.args;
                const long count = (long)rows * kHidden;
                a.group0 = agent0; a.groups = groups; a.M = rows; a.split_k = split; a.max_ctas = c->cur_ctas; a.am = sel_map(c);
                a.flags = 0; a.bias = nullptr;
                a.out = c->splitk_ws + (long)agent0 * c->splitk_group_stride;
                a.out_group_stride = c->splitk_group_stride; a.out_split_stride = count;
                LAUNCH(p.tag, st, launch_gemm(p.A, p.B, a, st));
                if (pend) { pend->split = split; pend->count = count; return GALA_OK; }
                LAUNCH(T_SPLITK, st, launch_splitk_reduce_act(c->splitk_ws + (long)agent0 * c->splitk_group_stride,
                                                              c->hid + (long)agent0 * B * kHidden, c->x + c->cl.fcb, dp, agent0,
                                                              count, kHidden, split, count, groups, c->splitk_group_stride,
                                                              B * kHidden, st));
            }
        }
        if (pend) return GALA_OK;
        HeadsArgs h{};
        h.rows = rows; h.H = kHidden; h.A = c->A;
        h.h = c->hid + (long)agent0 * B * kHidden; h.h_stride = B * kHidden; h.h_bf16 = 1;
        h.params = c->x + (long)agent0 * dp; h.p_stride = dp;
        h.piw = c->cl.piw; h.pib = c->cl.pib; h.vw = c->cl.vw; h.vb = c->cl.vb;
        h.logits = c->logits + (long)agent0 * B * c->A; h.logits_stride = B * c->A;
        h.values = c->values + (long)agent0 * B; h.values_stride = B;
        LAUNCH(T_HEADS_FWD, st, launch_heads_fwd(h, groups, st));
    } else {
        const int H = c->H;
        DenseArgs a{};
        a.rows = rows; a.in_dim = c->obs_dim; a.out_dim = H; a.act = 2;
        a.in = obs; a.in_bf16 = 0;
        a.W = c->x + (long)agent0 * dp + c->ml.w1; a.b = c->x + (long)agent0 * dp + c->ml.b1; a.w_stride = dp;
        a.out = c->h1 + (long)agent0 * B * H; a.out_stride = B * H; a.out_bf16 = 0;
        LAUNCH(T_DENSE_FWD, st, launch_dense_fwd(a, groups, st));
        DenseArgs b = a;
        b.in_dim = H;
        fill_batch(b.in, c->h1, B * H * 4, agent0, groups);
        b.W = c->x + (long)agent0 * dp + c->ml.w2; b.b = c->x + (long)agent0 * dp + c->ml.b2;
        b.out = c->h2 + (long)agent0 * B * H;
        LAUNCH(T_DENSE_FWD, st, launch_dense_fwd(b, groups, st));
        HeadsArgs h{};
        h.rows = rows; h.H = H; h.A = c->A;
        h.h = c->h2 + (long)agent0 * B * H; h.h_stride = B * H; h.h_bf16 = 0;
        h.params = c->x + (long)agent0 * dp; h.p_stride = dp;
        h.piw = c->ml.piw; h.pib = c->ml.pib; h.vw = c->ml.vw; h.vb = c->ml.vb;
        h.logits = c->logits + (long)agent0 * B * c->A; h.logits_stride = B * c->A;
        h.values = c->values + (long)agent0 * B; h.values_stride = B;
        LAUNCH(T_HEADS_FWD, st, launch_heads_fwd(h, groups, st));
    }
    return GALA_OK;
}

// Learner step for agents [agent0, agent0+groups): forward, returns/advantages/objective,
// backward into the flat gradient, global norm and clip coefficient.
int learn_range(gala_ctx* c, int agent0, int groups, const gala_rollout* ro, cudaStream_t st,
                cudaStream_t side = nullptr) {
    const long dp = c->d_pad, B = c->B, S = c->S;
    const int A = c->A;
    PtrBatch obs{}, acts{}, rews{}, dns{};
    for (int i = 0; i < groups; i++) {
        obs.p[i] = ro[i].obs; acts.p[i] = ro[i].actions; rews.p[i] = ro[i].rewards; dns.p[i] = ro[i].dones;
    }
    // Second stream of the synchronous mode: work that the chain forward -> loss -> data gradients does not
    // wait for.  `fork` makes it wait for what `st` has enqueued so far.
    cudaStream_t ws = side ? side : st;
    auto fork = [&]() -> int {
        if (!side) return GALA_OK;
        CK(cudaEventRecord(c->cur_fork, st));
        CK(cudaStreamWaitEvent(side, c->cur_fork, 0));
        return GALA_OK;
    };
    c->pending.n = 0;
    // forward pass and weight gradient of conv1 read the uint8 frames themselves; only the legacy products
    // need bf16 copies
    if (!c->conv && c->fused_mlp) {
        MlpFusedArgs m{};
        m.D = c->obs_dim; m.H = c->H; m.A = A; m.T = c->T; m.E = c->E; m.d = c->d; m.l = c->ml;
        m.gamma = c->hp.gamma; m.ent_coef = c->hp.ent_coef; m.vf_coef = c->hp.vf_coef; m.max_norm = c->hp.max_grad_norm;
        m.params = c->x + (long)agent0 * dp; m.p_stride = dp;
        m.obs = obs; m.actions = acts; m.rewards = rews; m.dones = dns;
        m.logits = c->logits + (long)agent0 * B * A; m.values = c->values + (long)agent0 * B;
        m.returns = c->returns + (long)agent0 * S; m.adv = c->adv + (long)agent0 * S;
        m.dlogits = c->dlogits + (long)agent0 * S * A; m.dvalues = c->dvalues + (long)agent0 * S;
        m.losses = c->losses + (long)agent0 * 4;
        m.h1_out = c->h1 + (long)agent0 * B * c->H; m.h2_out = c->h2 + (long)agent0 * B * c->H;
        m.grad = c->g + (long)agent0 * dp; m.g_stride = dp;
        m.norm = c->norm + agent0; m.clip = c->clip + agent0;
        m.partial = c->mlp_partial + (long)agent0 * kMlpMaxBlocks * mlp_fused_partial_stride(c->d);
        m.ticket = c->heads_ticket + agent0;
        LAUNCH(T_MLP_FUSED, st, launch_mlp_fused(m, groups, st));
        for (int i = 0; i < groups; i++) {
            Agent& ag = c->agents[sel_agent(c, agent0, i)];
            ag.pending = true;
            ag.frames += S;
        }
        return GALA_OK;
    }
    HiddenPending pend;
    const bool fused = c->conv && c->fused_heads;
    int r = forward(c, agent0, groups, obs, (int)B, st, c->legacy_conv ? st : nullptr, fused ? &pend : nullptr);
    if (r != GALA_OK) return r;
    LossArgs la{};
    la.T = c->T; la.E = c->E; la.A = A; la.B = B;
    la.gamma = c->hp.gamma; la.ent_coef = c->hp.ent_coef; la.vf_coef = c->hp.vf_coef;
    la.logits = c->logits + (long)agent0 * B * A; la.values = c->values + (long)agent0 * B;
    la.actions = acts; la.rewards = rews; la.dones = dns;
    la.returns = c->returns + (long)agent0 * S; la.adv = c->adv + (long)agent0 * S;
    la.dlogits = c->dlogits + (long)agent0 * S * A; la.dvalues = c->dvalues + (long)agent0 * S;
    la.losses = c->losses + (long)agent0 * 4;
    if (fused) {
        HeadsFusedArgs hf{};
        hf.T = c->T; hf.E = c->E; hf.A = A; hf.B = B;
        hf.gamma = c->hp.gamma; hf.ent_coef = c->hp.ent_coef; hf.vf_coef = c->hp.vf_coef;
        hf.hid = c->hid + (long)agent0 * B * kHidden; hf.hid_out = c->hid + (long)agent0 * B * kHidden;
        hf.h_stride = B * kHidden;
        if (pend.split > 1) {
            hf.partials = c->splitk_ws + (long)agent0 * c->splitk_group_stride;
            hf.split = pend.split; hf.split_stride = pend.count; hf.partial_group_stride = c->splitk_group_stride;
        }
        hf.params = c->x + (long)agent0 * dp; hf.p_stride = dp;
        hf.piw = c->cl.piw; hf.pib = c->cl.pib; hf.vw = c->cl.vw; hf.vb = c->cl.vb; hf.fcb = c->cl.fcb;
        hf.actions = acts; hf.rewards = rews; hf.dones = dns;
        hf.logits = c->logits + (long)agent0 * B * A; hf.values = c->values + (long)agent0 * B;
        hf.returns = la.returns; hf.adv = la.adv; hf.dlogits = la.dlogits; hf.dvalues = la.dvalues;
        hf.losses = la.losses;
        hf.dzv = c->dzv + (long)agent0 * S * 20;
        hf.dh = c->dh + (long)agent0 * S * kHidden; hf.dh_stride = S * kHidden;
        hf.loss_partial = c->heads_partial + (long)agent0 * c->E * 4;
        hf.ticket = c->heads_ticket + agent0;
        hf.am = sel_map(c);
        LAUNCH(T_HEADS_FUSED, st, launch_heads_fused(hf, groups, st));
    } else {
        LAUNCH(T_LOSS, st, launch_a2c_loss(la, groups, st));
    }

    HeadsBwdArgs hb{};
    hb.rows = (int)S; hb.A = A;
    hb.params = c->x + (long)agent0 * dp; hb.p_stride = dp;
    hb.dlogits = la.dlogits; hb.dlogits_stride = S * A;
    hb.dvalues = la.dvalues; hb.dvalues_stride = S;
    hb.grad = c->g + (long)agent0 * dp; hb.g_stride = dp;
    hb.am = sel_map(c);
    if (c->conv) {
        const int P[3] = {400, 81, 49};
        hb.H = kHidden; hb.act = 1;
        hb.h = c->hid + (long)agent0 * B * kHidden; hb.h_stride = B * kHidden; hb.h_bf16 = 1;
        hb.piw = c->cl.piw; hb.pib = c->cl.pib; hb.vw = c->cl.vw; hb.vb = c->cl.vb;
        hb.dpre = c->dh + (long)agent0 * S * kHidden; hb.dpre_stride = S * kHidden; hb.dpre_bf16 = 1;
        // The data gradients form a chain (heads -> hidden -> conv3 -> conv2); every weight gradient only needs
        // the dY of its own layer.  With a side stream the weight gradients (and the bias gradients) run beside
        // the chain.
        if ((r = fork()) != GALA_OK) return r;
        if (fused) {
            hb.dzv = c->dzv + (long)agent0 * S * 20;
            LAUNCH(T_HEADS_BWD, ws, launch_heads_wgrad_tiled(hb, groups, ws));
        } else {
            LAUNCH(T_HEADS_BWD, ws, launch_heads_wgrad(hb, groups, ws));
            LAUNCH(T_HEADS_BWD, st, launch_heads_dgrad(hb, groups, st));
        }
        if ((r = fork()) != GALA_OK) return r;
        if ((r = run_plan(c, c->fc_wgrad, agent0, groups, 0, ws)) != GALA_OK) return r;
        if ((r = run_plan(c, c->fc_dgrad, agent0, groups, 0, st)) != GALA_OK) return r;
        // The chain ends with conv2's data gradient, the second stream is still busy with weight gradients
        // then: conv1's weight gradient, its slice sum and the column sums follow the chain on `st`.
        const bool tail_on_chain = side && !c->legacy_conv;
        // ... the column sums on a third stream beside conv1's weight gradient (synchronous round only)
        const bool tail_third = tail_on_chain && st == c->main_stream && side == c->side_stream;
        for (int l = 2; l >= 0; l--) {
            if (l == 0 && tail_on_chain) {
                if ((r = flush_pending_reduces(c, agent0, groups, ws)) != GALA_OK) return r;
                if (tail_third) {   // the column sums need dh and dY1, both complete here
                    CK(cudaEventRecord(c->ev_tail_fork, st));
                    CK(cudaStreamWaitEvent(c->tail_stream, c->ev_tail_fork, 0));
                }
                if ((r = run_conv1_wgrad(c, agent0, groups, obs, st)) != GALA_OK) return r;
                if ((r = flush_pending_reduces(c, agent0, groups, st)) != GALA_OK) return r;
                break;
            }
            if ((r = fork()) != GALA_OK) return r;
            r = c->legacy_conv ? run_wgrad(c, c->wgrad[l], agent0, groups, ws)
                : l > 0        ? run_conv_wgrad(c, c->cwgrad[l], agent0, groups, ws)
                               : run_conv1_wgrad(c, agent0, groups, obs, ws);
            if (r != GALA_OK) return r;
            if (l > 0) {
                r = c->legacy_conv ? run_plan(c, c->dgrad[l], agent0, groups, 0, st)
                                   : run_conv(c, c->cdgrad[l], agent0, groups, (int)S, st);
                if (r != GALA_OK) return r;
            }
        }
        if ((r = flush_pending_reduces(c, agent0, groups, ws)) != GALA_OK) return r;
        // Bias gradients = column sums.  conv2's and conv3's come out of their weight-gradient kernels (summed from
        // the dY tiles while those are in shared memory), conv1's out of conv2's data gradient as slices per CTA
        // and warp that are added here; the hidden layer's, and in the legacy mode all four, are summed here.
        {
            ColsumJobs jobs{};
            jobs.j[0] = {c->dh + (long)agent0 * S * kHidden, S * kHidden, S, kHidden, c->cl.fcb};
            const int order[3] = {0, 1, 2};
            for (int k = 0; k < 3; k++) {
                const int l = order[k];
                jobs.j[1 + k] = {c->dy[l] + (long)agent0 * S * P[l] * kConvCout[l], S * P[l] * kConvCout[l], S * P[l],
                                 kConvCout[l], c->cl.b[l]};
            }
            cudaStream_t cs = tail_third ? c->tail_stream : tail_on_chain ? st : ws;
            if (!tail_on_chain && (r = fork()) != GALA_OK) return r;
            ColsumSlices sl{c->c1b + (long)agent0 * kConvBiasSliceStride, c->cl.b[0],
                            conv_grid((long)groups * S, c->cur_ctas), (int)S};
            // few samples: the slices' extra work in the epilogue is exposed and the column sums cost a launch's
            // latency either way, so conv1's bias gradient is summed from dY1 like the hidden layer's
            const bool slices = !c->legacy_conv && (long)groups * S >= c->c1b_min_samples;
            LAUNCH(T_COLSUM, cs, launch_colsum(jobs, c->legacy_conv ? 4 : slices ? 1 : 2, c->g + (long)agent0 * dp, dp,
                                               c->colsum_partial + (long)agent0 * kColsumJobs * kColsumChunks * 512,
                                               c->colsum_ticket + (long)agent0 * kColsumJobs, groups, cs,
                                               slices ? &sl : nullptr, c->cur_map));
        }
        if (side) {   // join: the gradient is complete when all streams are done
            CK(cudaEventRecord(c->cur_join, side));
            CK(cudaStreamWaitEvent(st, c->cur_join, 0));
            if (tail_third) {
                CK(cudaEventRecord(c->ev_tail_join, c->tail_stream));
                CK(cudaStreamWaitEvent(st, c->ev_tail_join, 0));
            }
        }
    } else {
        const int H = c->H;
        hb.H = H; hb.act = 2;
        hb.h = c->h2 + (long)agent0 * B * H; hb.h_stride = B * H; hb.h_bf16 = 0;
        hb.piw = c->ml.piw; hb.pib = c->ml.pib; hb.vw = c->ml.vw; hb.vb = c->ml.vb;
        hb.dpre = c->dpre2 + (long)agent0 * S * H; hb.dpre_stride = S * H; hb.dpre_bf16 = 0;
        LAUNCH(T_HEADS_BWD, st, launch_heads_dgrad(hb, groups, st));
        LAUNCH(T_HEADS_BWD, st, launch_heads_wgrad(hb, groups, st));
        DenseBwdArgs d2{};
        d2.rows = (int)S; d2.in_dim = H; d2.out_dim = H; d2.act_in = 2;
        fill_batch(d2.in, c->h1, B * H * 4, agent0, groups);
        d2.dpre = c->dpre2 + (long)agent0 * S * H; d2.dpre_stride = S * H;
        d2.W = c->x + (long)agent0 * dp + c->ml.w2; d2.w_stride = dp;
        d2.gW = c->g + (long)agent0 * dp + c->ml.w2; d2.gb = c->g + (long)agent0 * dp + c->ml.b2; d2.g_stride = dp;
        d2.din = c->dpre1 + (long)agent0 * S * H; d2.din_stride = S * H;
        LAUNCH(T_DENSE_BWD, st, launch_dense_bwd(d2, groups, st));
        c->launches++; c->tag_launches[T_DENSE_BWD]++;
        DenseBwdArgs d1{};
        d1.rows = (int)S; d1.in_dim = c->obs_dim; d1.out_dim = H; d1.act_in = 0;
        d1.in = obs;
        d1.dpre = c->dpre1 + (long)agent0 * S * H; d1.dpre_stride = S * H;
        d1.W = c->x + (long)agent0 * dp + c->ml.w1; d1.w_stride = dp;
        d1.gW = c->g + (long)agent0 * dp + c->ml.w1; d1.gb = c->g + (long)agent0 * dp + c->ml.b1; d1.g_stride = dp;
        d1.din = nullptr;
        LAUNCH(T_DENSE_BWD, st, launch_dense_bwd(d1, groups, st));
    }
    NormKnown kn{};
    if (c->conv) {   // the hidden layer's weight gradient left the sums of squares of its 32 x 32 blocks behind
        kn.n_partials = (long)(kHidden / 128) * ((kFeat + 127) / 128) * 16;
        kn.off = c->cl.fcw; kn.count = (long)kHidden * kFeat;
        kn.partial = c->fc_sq + (long)agent0 * kn.n_partials; kn.partial_group_stride = kn.n_partials;
    }
    LAUNCH(T_GRAD_NORM, st, launch_grad_norm(c->g, c->d, dp, agent0, groups, c->hp.max_grad_norm, c->norm_partial, c->norm_ticket,
                            c->norm, c->clip, st, c->conv ? &kn : nullptr, c->cur_map));
    for (int i = 0; i < groups; i++) {
        Agent& ag = c->agents[sel_agent(c, agent0, i)];
        ag.pending = true;
        ag.frames += S;
    }
    return GALA_OK;
}

// learn_range through the graph cache.  First time a set of rollout buffers is seen: direct launches.  Second
// time: the same launches are captured into a graph, which is instantiated and launched.  From then on: one
// graph launch.  Per-class timing of a kernel inside the step and the legacy products go the direct way.
constexpr size_t kMaxStepGraphs = 512;
int learn_range_cached(gala_ctx* c, int agent0, int groups, const gala_rollout* ro, cudaStream_t st,
                       cudaStream_t side = nullptr) {
    // per-class timing brackets launches with events: not inside a graph (the optimiser / gossip pass and the
    // sampling kernel lie outside this step, so timing only those does not matter)
    const unsigned long long outside = (1ull << T_SWEEP_SYNC) | (1ull << T_SWEEP_AGENT) | (1ull << T_SAMPLE);
    if (c->use_graphs < (side ? 1 : 2) || (c->profile_mask & ~outside) != 0 || c->legacy_conv)
        return learn_range(c, agent0, groups, ro, st, side);
    std::vector<const void*> key;
    key.reserve(6 + 4 * (size_t)groups);
    key.push_back(st); key.push_back(side);
    key.push_back(reinterpret_cast<const void*>((uintptr_t)agent0));
    key.push_back(reinterpret_cast<const void*>((uintptr_t)groups));
    key.push_back(reinterpret_cast<const void*>((uintptr_t)c->cur_ctas));
    for (int i = 0; i < groups; i++) {
        key.push_back(ro[i].obs); key.push_back(ro[i].actions); key.push_back(ro[i].rewards); key.push_back(ro[i].dones);
    }
    StepGraph* g = nullptr;
    for (StepGraph& e : c->graphs)
        if (e.key == key) { g = &e; break; }
    if (!g) {
        if (c->graphs.size() < kMaxStepGraphs) { c->graphs.emplace_back(); c->graphs.back().key = std::move(key); }
        return learn_range(c, agent0, groups, ro, st, side);
    }
    if (g->failed) return learn_range(c, agent0, groups, ro, st, side);
    if (!g->exec) {
        if (cudaStreamBeginCapture(st, cudaStreamCaptureModeRelaxed) != cudaSuccess) {
            (void)cudaGetLastError();
            g->failed = true;
            return learn_range(c, agent0, groups, ro, st, side);
        }
        const long long l0 = c->launches;
        long long t0[T_COUNT];
        for (int k = 0; k < T_COUNT; k++) t0[k] = c->tag_launches[k];
        const int r = learn_range(c, agent0, groups, ro, st, side);   // enqueues nothing: the launches are recorded
        cudaGraph_t graph = nullptr;
        cudaError_t e = cudaStreamEndCapture(st, &graph);
        if (r == GALA_OK && e == cudaSuccess && graph) e = cudaGraphInstantiate(&g->exec, graph, 0);
        if (graph) cudaGraphDestroy(graph);
        if (r != GALA_OK || e != cudaSuccess || !g->exec) {
            (void)cudaGetLastError();
            g->failed = true; g->exec = nullptr;
            c->launches = l0;
            for (int k = 0; k < T_COUNT; k++) c->tag_launches[k] = t0[k];
            if (r != GALA_OK) return r;
            for (int i = 0; i < groups; i++) c->agents[agent0 + i].frames -= c->S;   // counted again below
            return learn_range(c, agent0, groups, ro, st, side);
        }
        g->launches = c->launches - l0;
        for (int k = 0; k < T_COUNT; k++) g->tag_launches[k] = c->tag_launches[k] - t0[k];
        CK(cudaGraphLaunch(g->exec, st));
        return GALA_OK;   // learn_range has already updated the host-side state for this step
    }
    CK(cudaGraphLaunch(g->exec, st));
    c->launches += g->launches;
    for (int k = 0; k < T_COUNT; k++) c->tag_launches[k] += g->tag_launches[k];
    for (int i = 0; i < groups; i++) {
        c->agents[agent0 + i].pending = true;
        c->agents[agent0 + i].frames += c->S;
    }
    return GALA_OK;
}

// Newest snapshot version of agent j that a sweep enqueued now on stream `st` may read (0: none): its writing
// sweep has completed, or it was enqueued earlier on the same stream and so completes before the reader runs
// (the grouped calls share their streams; an agent's own stream carries no other agent's sweeps).
long long usable_version(gala_ctx* c, int j, cudaStream_t st) {
    Agent& a = c->agents[j];
    for (long long w = a.version; w > 0 && w >= a.version - 1; w--)
        if (a.pub_stream[w % kSnapSlots] == st || cudaEventQuery(a.pub_event[w % kSnapSlots]) == cudaSuccess) return w;
    return 0;
}

// What one agent's optimiser / gossip step will do, decided on the host when it is enqueued.
struct SweepPlan {
    int np = 0;                    // in-peers of the agent's current round
    int peers[2] = {0, 0};
    long long vers[2] = {0, 0};    // snapshot version taken from each
    bool fresh = false;            // a newer completed snapshot than the one last consumed exists for every in-peer
    bool waited = false;           // ... after a wait forced by the staleness bound
    long long w = 0;               // version the agent publishes
    int slot = 0;                  // and its slot
};

// Decides (and, under the staleness bound, waits on the host); changes nothing in the context.
int plan_sweep(gala_ctx* c, int i, bool try_mix, cudaStream_t st, SweepPlan* sp) {
    Agent& ag = c->agents[i];
    int off[2] = {0, 0};
    sp->np = try_mix ? topo_offsets(c->topo, c->n, ag.round, off) : 0;
    sp->fresh = sp->np > 0;
    for (int j = 0; j < sp->np; j++) {
        sp->peers[j] = ((i - off[j]) % c->n + c->n) % c->n;
        sp->vers[j] = usable_version(c, sp->peers[j], st);
        if (sp->vers[j] <= ag.consumed[sp->peers[j]]) sp->fresh = false;
    }
    // Staleness bound (Sec. 3): if more than tau local iterations have passed since this agent last
    // averaged, it waits for its in-peers' newest snapshots instead of going on alone.  The wait is a
    // host wait with a deadline; only snapshots that are already enqueued can complete, so if an
    // in-peer has nothing newer on its stream the call gives up at once.
    if (try_mix && sp->np > 0 && !sp->fresh && c->hp.staleness_tau >= 0 && ag.since_mix > c->hp.staleness_tau) {
        for (int j = 0; j < sp->np; j++) {
            Agent& pj = c->agents[sp->peers[j]];
            if (pj.version <= ag.consumed[sp->peers[j]])
                return fail(c, GALA_ETIMEOUT, "agent %d: %lld iterations without a message and in-peer %d has published "
                            "nothing newer (tau = %d)", i, ag.since_mix, sp->peers[j], c->hp.staleness_tau);
        }
        const auto t0 = std::chrono::steady_clock::now();
        for (int j = 0; j < sp->np; j++) {
            Agent& pj = c->agents[sp->peers[j]];
            for (;;) {
                cudaError_t e = cudaEventQuery(pj.pub_event[pj.version % kSnapSlots]);
                if (e == cudaSuccess) break;
                if (e != cudaErrorNotReady) return fail(c, GALA_ECUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
                const auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(std::chrono::steady_clock::now() - t0).count();
                if (ms >= c->stale_timeout_ms)
                    return fail(c, GALA_ETIMEOUT, "agent %d: in-peer %d's snapshot still not complete after %d ms", i,
                                sp->peers[j], c->stale_timeout_ms);
                std::this_thread::sleep_for(std::chrono::microseconds(20));
            }
            sp->vers[j] = pj.version;
        }
        sp->fresh = true;
        sp->waited = true;
    }
    sp->w = ag.version + 1;
    sp->slot = (int)(sp->w % kSnapSlots);
    return GALA_OK;
}

// Pairwise back-pressure: sweeps that may still read the slot the agent is about to overwrite go first.
// `st` is the stream the agent's new sweep goes to; readers whose latest sweep sits on the same stream are
// ordered already.
int sweep_backpressure(gala_ctx* c, int i, const SweepPlan& sp, cudaStream_t st) {
    Agent& ag = c->agents[i];
    for (int r : ag.slot_readers[sp.slot]) {
        Agent& rd = c->agents[r];
        if (rd.version > 0 && rd.sweep_stream != st) CK(cudaStreamWaitEvent(st, rd.pub_event[rd.version % kSnapSlots], 0));
    }
    ag.slot_readers[sp.slot].clear();
    return GALA_OK;
}

// Host-side record of a sweep that has been enqueued on `st` (its completion event recorded by the caller).
void commit_sweep(gala_ctx* c, int i, const SweepPlan& sp, cudaStream_t st) {
    Agent& ag = c->agents[i];
    if (sp.fresh) {
        for (int j = 0; j < sp.np; j++) {
            Agent& pj = c->agents[sp.peers[j]];
            pj.slot_readers[sp.vers[j] % kSnapSlots].push_back(i);
            const long long stale = pj.version - sp.vers[j];
            ag.stale_sum += stale;
            if (stale > ag.stale_max) ag.stale_max = stale;
            ag.consumed[sp.peers[j]] = sp.vers[j];
        }
        ag.mixes++;
        ag.since_mix = 0;
    } else if (sp.np > 0) {
        ag.skipped++;
        ag.since_mix++;
    }
    if (sp.waited) ag.stale_waits++;
    ag.version = sp.w;
    ag.sweep_stream = st;
    ag.pub_stream[sp.slot] = st;
    ag.pending = false;
    ag.last_n = sp.np; ag.last_mixed = sp.fresh ? 1 : 0;
    for (int j = 0; j < 2; j++) { ag.last_peers[j] = sp.peers[j]; ag.last_versions[j] = sp.fresh ? sp.vers[j] : 0; }
}

// Orders the agent's own stream behind the group launches that touched the agent, before a per-agent call
// enqueues on it.
int own_stream_begin(gala_ctx* c, Agent& ag) {
    if (ag.group_lane >= 0) {
        CK(cudaStreamWaitEvent(ag.stream, c->glane[ag.group_lane].done, 0));
        ag.group_lane = -1;
    }
    ag.dirty = true;
    return GALA_OK;
}

// Optimiser step + publication (+ conditional average) for one agent on its stream.
int sweep_agent(gala_ctx* c, int i, bool try_mix) {
    Agent& ag = c->agents[i];
    const long dp = c->d_pad;
    SweepPlan sp;
    int r = plan_sweep(c, i, try_mix, ag.stream, &sp);
    if (r != GALA_OK) return r;
    if ((r = own_stream_begin(c, ag)) != GALA_OK) return r;
    if ((r = sweep_backpressure(c, i, sp, ag.stream)) != GALA_OK) return r;
    const float* p0 = nullptr;
    const float* p1 = nullptr;
    if (sp.fresh)
        for (int j = 0; j < sp.np; j++) {
            const float* ptr = c->snap + ((long)sp.peers[j] * kSnapSlots + sp.vers[j] % kSnapSlots) * dp;
            if (j == 0) p0 = ptr; else p1 = ptr;
        }
    SweepHp hp{c->hp.lr, c->hp.rms_alpha, c->hp.rms_eps};
    LAUNCH(T_SWEEP_AGENT, ag.stream, launch_sweep_agent(c->x + (long)i * dp, ag.pending ? c->g + (long)i * dp : nullptr, c->v + (long)i * dp,
                              c->snap + ((long)i * kSnapSlots + sp.slot) * dp, p0, p1, sp.fresh ? sp.np : 0, c->clip + i,
                              c->conv ? c->shadow + (long)i * dp : nullptr, dp, hp, ag.stream));
    CK(cudaEventRecord(ag.pub_event[sp.slot], ag.stream));
    commit_sweep(c, i, sp, ag.stream);
    return GALA_OK;
}

// A group lane becomes ordered behind everything that was enqueued for the listed agents elsewhere: work on their
// own streams (per-agent calls, the tail of a synchronous round) and launch sets on the other lane.
int lane_acquire(gala_ctx* c, int lane, const int* agents, int m) {
    gala_ctx::Lane& L = c->glane[lane];
    bool other = false;
    for (int k = 0; k < m; k++) {
        Agent& ag = c->agents[agents[k]];
        if (ag.dirty) {
            CK(cudaEventRecord(ag.fence, ag.stream));
            CK(cudaStreamWaitEvent(L.st, ag.fence, 0));
            ag.dirty = false;
        }
        if (ag.group_lane >= 0 && ag.group_lane != lane) other = true;
    }
    if (other) CK(cudaStreamWaitEvent(L.st, c->glane[lane ^ 1].done, 0));
    return GALA_OK;
}
int lane_release(gala_ctx* c, int lane, const int* agents, int m) {
    CK(cudaEventRecord(c->glane[lane].done, c->glane[lane].st));
    for (int k = 0; k < m; k++) c->agents[agents[k]].group_lane = lane;
    return GALA_OK;
}

// Optimiser step + publication (+ conditional average) for a list of distinct agents on a group lane, one
// launch per kBatch agents.  All decisions are taken before anything is enqueued or recorded, so an agent of the
// list never counts a snapshot of the same call as complete.
int sweep_group(gala_ctx* c, int lane, const int* agents, int m, bool try_mix) {
    gala_ctx::Lane& L = c->glane[lane];
    const long dp = c->d_pad;
    std::vector<SweepPlan> plans((size_t)m);
    for (int k = 0; k < m; k++) {
        int r = plan_sweep(c, agents[k], try_mix, L.st, &plans[k]);
        if (r != GALA_OK) return r;
    }
    for (int k = 0; k < m; k++) {
        int r = sweep_backpressure(c, agents[k], plans[k], L.st);
        if (r != GALA_OK) return r;
    }
    for (int k0 = 0; k0 < m; k0 += kBatch) {
        const int cnt = m - k0 < kBatch ? m - k0 : kBatch;
        SweepManyArgs a{};
        a.x = c->x; a.g = c->g; a.v = c->v; a.snap = c->snap; a.shadow = c->conv ? c->shadow : nullptr; a.clip = c->clip;
        a.d_pad = dp; a.hp = SweepHp{c->hp.lr, c->hp.rms_alpha, c->hp.rms_eps}; a.error_word = c->error_word;
        a.n_items = cnt;
        for (int e = 0; e < cnt; e++) {
            const int i = agents[k0 + e];
            const SweepPlan& sp = plans[k0 + e];
            SweepItem& it = a.it[e];
            it.x_row = i;
            it.out_row = i * kSnapSlots + sp.slot;
            it.p_row[0] = it.p_row[1] = -1;
            if (sp.fresh)
                for (int j = 0; j < sp.np; j++) it.p_row[j] = sp.peers[j] * kSnapSlots + (int)(sp.vers[j] % kSnapSlots);
            if (c->agents[i].pending) a.has_grad[e >> 5] |= 1u << (e & 31);
        }
        LAUNCH(T_SWEEP_AGENT, L.st, launch_sweep_many(a, L.st));
    }
    for (int k = 0; k < m; k++) {
        CK(cudaEventRecord(c->agents[agents[k]].pub_event[plans[k].slot], L.st));
        commit_sweep(c, agents[k], plans[k], L.st);
    }
    return GALA_OK;
}

int host_wait(gala_ctx* c, cudaStream_t st, int timeout_ms) {
    if (timeout_ms < 0) {
        CK(cudaStreamSynchronize(st));
        return GALA_OK;
    }
    auto t0 = std::chrono::steady_clock::now();
    for (;;) {
        cudaError_t e = cudaStreamQuery(st);
        if (e == cudaSuccess) return GALA_OK;
        if (e != cudaErrorNotReady) return fail(c, GALA_ECUDA, "cudaStreamQuery: %s", cudaGetErrorString(e));
        auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(std::chrono::steady_clock::now() - t0).count();
        if (ms >= timeout_ms) return fail(c, GALA_ETIMEOUT, "work still running after %d ms", timeout_ms);
        std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
}

// Copy into device memory that is complete when the call returns.  A plain cudaMemcpy from pageable host memory may
// return while its last piece is still on the way, and the library's streams are non-blocking, i.e. not ordered
// behind the default stream that copy runs on: a kernel launched right after it could read the old contents.
int copy_in(gala_ctx* c, void* dst, const void* src, size_t bytes, cudaStream_t st) {
    CK(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, st));
    CK(cudaStreamSynchronize(st));
    return GALA_OK;
}

int check_error_word(gala_ctx* c) {
    int w = 0;
    CK(cudaMemcpy(&w, c->error_word, sizeof w, cudaMemcpyDeviceToHost));
    if (w) {
        int z = 0;
        (void)copy_in(c, c->error_word, &z, sizeof z, c->main_stream);
        // 1 hidden-layer product, 2 / 3 optimiser passes, 10.. convolution variant, 21 / 22 conv2 / conv3 weight
        // gradient, 30 conv1 weight gradient
        return fail(c, GALA_ECUDA, "a bounded device-side wait ran out (kernel code %d)", w);
    }
    return GALA_OK;
}

bool valid_agent(const gala_ctx* c, int a) { return c && a >= 0 && a < c->n; }

// Host wait for everything that was enqueued for the agent, wherever it went: the synchronous stream, the lane
// of the last grouped call that listed it, its own stream.
int settle_agent(gala_ctx* c, int agent) {
    Agent& ag = c->agents[agent];
    CK(cudaStreamSynchronize(c->main_stream));
    if (ag.group_lane >= 0) CK(cudaStreamSynchronize(c->glane[ag.group_lane].st));
    CK(cudaStreamSynchronize(ag.stream));
    return GALA_OK;
}

}  // namespace

// ====================================================================== C ABI
extern "C" {

int gala_create(int n_agents, const gala_topology* topo, const gala_net_spec* net, const gala_hparams* hp,
                gala_ctx** out) {
    if (!out) return GALA_EINVAL;
    *out = nullptr;
    if (!topo || !net || !hp) return GALA_EINVAL;
    if (n_agents < 1 || n_agents > 256) return GALA_EINVAL;
    if (topo->kind != GALA_TOPO_RING && topo->kind != GALA_TOPO_EXP && topo->kind != GALA_TOPO_COMPLETE) return GALA_EINVAL;
    if (topo->kind != GALA_TOPO_COMPLETE && (topo->peers < 1 || topo->peers > 2)) return GALA_EINVAL;
    if (net->kind != GALA_NET_MLP && net->kind != GALA_NET_CONV) return GALA_EINVAL;
    if (net->n_actions < 2 || net->n_actions > 32) return GALA_EINVAL;
    if (hp->n_envs < 1 || hp->n_steps < 1) return GALA_EINVAL;
    if (!(hp->rms_eps > 0.0f) || !(hp->lr >= 0.0f) || hp->rms_alpha < 0.0f || hp->rms_alpha > 1.0f) return GALA_EINVAL;
    if (net->kind == GALA_NET_MLP && (net->obs_dim < 1 || net->obs_dim > 4096 || net->hidden < 1 || net->hidden > 1024))
        return GALA_EINVAL;
    if (net->kind == GALA_NET_CONV && net->gemm_dtype != 1) return GALA_EINVAL;
    if (net->kind == GALA_NET_MLP && net->gemm_dtype != 0) return GALA_EINVAL;

    gala_ctx* c = new (std::nothrow) gala_ctx();
    if (!c) return GALA_ENOMEM;
    *out = c;  // handed out even on failure so that gala_last_error can explain; gala_destroy frees it
    c->n = n_agents; c->topo = *topo; c->net = *net; c->hp = *hp;
    c->conv = net->kind == GALA_NET_CONV;
    c->T = hp->n_steps; c->E = hp->n_envs; c->A = net->n_actions;
    c->B = (long)(c->T + 1) * c->E; c->S = (long)c->T * c->E;
    const int A = c->A;
    long off = 0;
    if (c->conv) {
        for (int l = 0; l < 3; l++) {
            c->cl.w[l] = off; off += (long)kConvCout[l] * kConvKK[l];
            c->cl.b[l] = off; off += kConvCout[l];
        }
        c->cl.fcw = off; off += (long)kHidden * kFeat;
        c->cl.fcb = off; off += kHidden;
        c->cl.piw = off; off += (long)A * kHidden;
        c->cl.pib = off; off += A;
        c->cl.vw = off; off += kHidden;
        c->cl.vb = off; off += 1;
        c->H = kHidden;
    } else {
        const int H = net->hidden, D = net->obs_dim;
        c->H = H; c->obs_dim = D;
        c->ml.w1 = off; off += (long)H * D;
        c->ml.b1 = off; off += H;
        c->ml.w2 = off; off += (long)H * H;
        c->ml.b2 = off; off += H;
        c->ml.piw = off; off += (long)A * H;
        c->ml.pib = off; off += A;
        c->ml.vw = off; off += H;
        c->ml.vb = off; off += 1;
    }
    c->d = off;
    c->d_pad = (off + 1023) / 1024 * 1024;
    const long dp = c->d_pad, B = c->B, S = c->S;
    const int n = c->n;

    CK(cudaStreamCreateWithFlags(&c->main_stream, cudaStreamNonBlocking));
    CK(cudaEventCreateWithFlags(&c->main_event, cudaEventDisableTiming));
    CK(cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking));
    CK(cudaStreamCreateWithFlags(&c->tail_stream, cudaStreamNonBlocking));
    CK(cudaEventCreateWithFlags(&c->ev_tail_fork, cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&c->ev_tail_join, cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming));
    c->cur_fork = c->ev_fork; c->cur_join = c->ev_join;
    for (gala_ctx::Lane& L : c->glane) {
        CK(cudaStreamCreateWithFlags(&L.st, cudaStreamNonBlocking));
        CK(cudaStreamCreateWithFlags(&L.side, cudaStreamNonBlocking));
        CK(cudaEventCreateWithFlags(&L.fork, cudaEventDisableTiming));
        CK(cudaEventCreateWithFlags(&L.join, cudaEventDisableTiming));
        CK(cudaEventCreateWithFlags(&L.done, cudaEventDisableTiming));
    }
    c->agents.resize(n);
    for (int i = 0; i < n; i++) {
        Agent& a = c->agents[i];
        CK(cudaStreamCreateWithFlags(&a.lib_stream, cudaStreamNonBlocking));
        a.stream = a.lib_stream;
        for (int s = 0; s < kSnapSlots; s++) CK(cudaEventCreateWithFlags(&a.pub_event[s], cudaEventDisableTiming));
        CK(cudaEventCreateWithFlags(&a.fence, cudaEventDisableTiming));
        a.consumed.assign(n, 0);
    }
    ALLOC(c->x, (size_t)n * dp); ALLOC(c->g, (size_t)n * dp); ALLOC(c->v, (size_t)n * dp);
    ALLOC(c->snap, (size_t)n * kSnapSlots * dp);
    ALLOC(c->clip, n); ALLOC(c->norm, n); ALLOC(c->losses, (size_t)n * 4);
    ALLOC(c->norm_partial, (size_t)n * kNormChunks); ALLOC(c->norm_ticket, n);
    ALLOC(c->error_word, 1);
    ALLOC(c->cons_partial, 592); ALLOC(c->cons_out, 1); ALLOC(c->cons_ticket, 1);
    ALLOC(c->upd_partial, (size_t)n * kUpdateNormChunks); ALLOC(c->upd_out, 1); ALLOC(c->upd_ticket, 1);
    ALLOC(c->logits, (size_t)n * B * A); ALLOC(c->values, (size_t)n * B);
    ALLOC(c->returns, (size_t)n * S); ALLOC(c->adv, (size_t)n * S);
    ALLOC(c->dlogits, (size_t)n * S * A); ALLOC(c->dvalues, (size_t)n * S);
    {   // clip coefficients start at 1
        std::vector<float> ones(n, 1.0f);
        int r = copy_in(c, c->clip, ones.data(), n * sizeof(float), c->main_stream);
        if (r != GALA_OK) return r;
    }
    if (c->conv) {
        const int P[3] = {400, 81, 49};
        CK(gemm_init());
        CK(conv_init());
        CK(wgrad_init());
        CK(wgrad1_init());
#ifdef GALA_CROSS_CHECK
        // Only in the cross-check build of the library (libgala_check.so, loaded by one test): the previous generation
        // of the convolution products, one tensor copy per kernel offset, as an independent second implementation.
        c->legacy_conv = getenv("GALA_CONV_LEGACY") != nullptr;
#endif
        if (n >= 5) c->agent_ctas = sm_count() * 8 / n < 32 ? 32 : sm_count() * 8 / n;   // measured on 64 agents: 32 beats 16 and 64
        c->fused_heads = heads_fused_supported(c->T, c->E, c->A, kHidden) && getenv("GALA_HEADS_UNFUSED") == nullptr;
        ALLOC(c->heads_partial, (size_t)n * c->E * 4); ALLOC(c->heads_ticket, n);
        ALLOC(c->dzv, (size_t)n * S * 20);
        c->fc_bn = c->B >= 256 ? 256 : 128;
        if (const char* e = getenv("GALA_FC_BN")) { const int v = atoi(e); if (v == 128 || v == 256) c->fc_bn = v; }
        ALLOC(c->fc_sq, (size_t)n * (kHidden / 128) * ((kFeat + 127) / 128) * 16);
        ALLOC(c->c1b, (size_t)n * kConvBiasSliceStride);
        if (const char* e = getenv("GALA_C1B_SLICES")) c->c1b_min_samples = atoi(e) ? 0 : (1L << 60);
        ALLOC(c->shadow, (size_t)n * dp);
        ALLOC(c->colsum_partial, (size_t)n * kColsumJobs * kColsumChunks * 512); ALLOC(c->colsum_ticket, (size_t)n * kColsumJobs);
        for (int l = 0; l < 3; l++) {
            ALLOC(c->act[l], (size_t)n * B * P[l] * kConvCout[l]);
            ALLOC(c->gate[l], (size_t)n * B * P[l] * kConvCout[l] / 32);
            ALLOC(c->dy[l], (size_t)n * S * P[l] * kConvCout[l]);
        }
        ALLOC(c->frames, (size_t)n * B * kFramePix);
        ALLOC(c->hid, (size_t)n * B * kHidden);
        ALLOC(c->dh, (size_t)n * S * kHidden);
        // slices of conv3 (also the hidden layer's split-K partial sums), conv2, conv1 weight gradients
        c->splitk_region[2] = 0;
        c->splitk_region[1] = (long)c->max_split * 64 * 576;
        c->splitk_region[0] = c->splitk_region[1] + (long)c->max_split * 64 * 512;
        c->bias_region[0] = c->splitk_region[0] + (long)c->max_split * 32 * 256;
        c->bias_region[1] = c->bias_region[0] + (long)c->max_split * 64;
        c->bias_region[2] = c->bias_region[1] + (long)c->max_split * 64;
        c->splitk_group_stride = c->bias_region[2] + (long)c->max_split * 64;
        ALLOC(c->splitk_ws, (size_t)n * c->splitk_group_stride);
        int r = build_plans(c);
        if (r != GALA_OK) return r;
    } else {
        const int H = c->H;
        ALLOC(c->h1, (size_t)n * B * H); ALLOC(c->h2, (size_t)n * B * H);
        ALLOC(c->dpre1, (size_t)n * S * H); ALLOC(c->dpre2, (size_t)n * S * H);
        c->fused_mlp = mlp_fused_supported(c->obs_dim, H, A, c->T, c->E, c->d) && getenv("GALA_MLP_UNFUSED") == nullptr;
        ALLOC(c->mlp_partial, (size_t)n * kMlpMaxBlocks * mlp_fused_partial_stride(c->d)); ALLOC(c->heads_ticket, n);
    }
    // initial parameters: uniform(-1,1)/sqrt(fan_in), biases included
    {
        std::vector<float> host((size_t)dp, 0.0f);
        for (int i = 0; i < n; i++) {
            const uint64_t ag = hp->identical_init ? 0 : (uint64_t)i;
            if (i == 0 || !hp->identical_init) {
                if (c->conv) {
                    for (int l = 0; l < 3; l++) {
                        init_tensor(host.data(), c->cl.w[l], (long)kConvCout[l] * kConvKK[l], kConvKK[l], hp->seed, ag);
                        init_tensor(host.data(), c->cl.b[l], kConvCout[l], kConvKK[l], hp->seed, ag);
                    }
                    init_tensor(host.data(), c->cl.fcw, (long)kHidden * kFeat, kFeat, hp->seed, ag);
                    init_tensor(host.data(), c->cl.fcb, kHidden, kFeat, hp->seed, ag);
                    init_tensor(host.data(), c->cl.piw, (long)A * kHidden, kHidden, hp->seed, ag);
                    init_tensor(host.data(), c->cl.pib, A, kHidden, hp->seed, ag);
                    init_tensor(host.data(), c->cl.vw, kHidden, kHidden, hp->seed, ag);
                    init_tensor(host.data(), c->cl.vb, 1, kHidden, hp->seed, ag);
                } else {
                    const int H = c->H, D = c->obs_dim;
                    init_tensor(host.data(), c->ml.w1, (long)H * D, D, hp->seed, ag);
                    init_tensor(host.data(), c->ml.b1, H, D, hp->seed, ag);
                    init_tensor(host.data(), c->ml.w2, (long)H * H, H, hp->seed, ag);
                    init_tensor(host.data(), c->ml.b2, H, H, hp->seed, ag);
                    init_tensor(host.data(), c->ml.piw, (long)A * H, H, hp->seed, ag);
                    init_tensor(host.data(), c->ml.pib, A, H, hp->seed, ag);
                    init_tensor(host.data(), c->ml.vw, H, H, hp->seed, ag);
                    init_tensor(host.data(), c->ml.vb, 1, H, hp->seed, ag);
                }
            }
            int r = copy_in(c, c->x + (long)i * dp, host.data(), dp * sizeof(float), c->main_stream);
            if (r != GALA_OK) return r;
        }
        if (c->conv) {
            LAUNCH(T_CAST, c->main_stream, launch_cast_bf16(c->x, c->shadow, (long)n * dp, c->main_stream));
            CK(cudaStreamSynchronize(c->main_stream));
        }
    }
    CK(cudaDeviceSynchronize());
    return GALA_OK;
}

int gala_destroy(gala_ctx* c) {
    if (!c) return GALA_EINVAL;
    cudaDeviceSynchronize();
    for (Agent& a : c->agents) {
        if (a.lib_stream) cudaStreamDestroy(a.lib_stream);
        for (int s = 0; s < kSnapSlots; s++) if (a.pub_event[s]) cudaEventDestroy(a.pub_event[s]);
        if (a.fence) cudaEventDestroy(a.fence);
    }
    for (StepGraph& g : c->graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
    for (Agent& a : c->agents) if (a.loop_graph.exec) cudaGraphExecDestroy(a.loop_graph.exec);
    if (c->la_graph.exec) cudaGraphExecDestroy(c->la_graph.exec);
    for (gala_ctx::Lane& L : c->glane) {
        if (L.st) cudaStreamDestroy(L.st);
        if (L.side) cudaStreamDestroy(L.side);
        if (L.fork) cudaEventDestroy(L.fork);
        if (L.join) cudaEventDestroy(L.join);
        if (L.done) cudaEventDestroy(L.done);
    }
    if (c->side_stream) cudaStreamDestroy(c->side_stream);
    if (c->tail_stream) cudaStreamDestroy(c->tail_stream);
    if (c->ev_tail_fork) cudaEventDestroy(c->ev_tail_fork);
    if (c->ev_tail_join) cudaEventDestroy(c->ev_tail_join);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    if (c->main_stream) cudaStreamDestroy(c->main_stream);
    if (c->main_event) cudaEventDestroy(c->main_event);
    for (auto& t : c->timed) { cudaEventDestroy(t.beg); cudaEventDestroy(t.end); }
    for (auto& e : c->event_pool) { cudaEventDestroy(e.first); cudaEventDestroy(e.second); }
    for (void* p : c->allocs) cudaFree(p);
    delete c;
    return GALA_OK;
}

int gala_act(gala_ctx* c, int agent, const void* obs, const float* uniforms, int* actions, float* values) {
    if (!valid_agent(c, agent) || !obs) return fail(c, GALA_EINVAL, "gala_act: bad agent or null obs");
    if (actions && !uniforms) return fail(c, GALA_EINVAL, "gala_act: actions requested without uniforms");
    Agent& ag = c->agents[agent];
    PtrBatch pb{};
    pb.p[0] = obs;
    int r = own_stream_begin(c, ag);
    if (r != GALA_OK) return r;
    c->cur_ctas = c->agent_ctas;
    r = forward(c, agent, 1, pb, c->E, ag.stream, c->legacy_conv ? ag.stream : nullptr);
    c->cur_ctas = 0;
    if (r != GALA_OK) return r;
    if (actions)
        LAUNCH(T_SAMPLE, ag.stream, launch_sample(c->logits + (long)agent * c->B * c->A, uniforms, actions, c->E, c->A, ag.stream));
    if (values)
        CK(cudaMemcpyAsync(values, c->values + (long)agent * c->B, c->E * sizeof(float), cudaMemcpyDeviceToDevice,
                           ag.stream));
    return GALA_OK;
}

// Rollout buffers of the closed loops, for all agents at once (the lockstep loop addresses them by stride).
static int ensure_loop_buffers(gala_ctx* c) {
    if (c->la_obs) return GALA_OK;
    const int T = c->T, E = c->E, n = c->n;
    const long obs_bytes = c->conv ? kFramePix : (long)c->obs_dim * 4;
    const size_t per_obs = (size_t)(T + 1) * E * obs_bytes, TE = (size_t)T * E;
    uint8_t* ob = nullptr;
    ALLOC(ob, (size_t)n * per_obs);
    ALLOC(c->la_actions, n * TE); ALLOC(c->la_rewards, n * TE); ALLOC(c->la_dones, n * TE);
    ALLOC(c->la_uniforms, (size_t)n * E); ALLOC(c->la_steps, n);
    for (int i = 0; i < n; i++) {
        Agent& ag = c->agents[i];
        ag.loop_obs = ob + i * per_obs;
        ag.loop_actions = c->la_actions + i * TE; ag.loop_rewards = c->la_rewards + i * TE;
        ag.loop_dones = c->la_dones + i * TE; ag.loop_uniforms = c->la_uniforms + (size_t)i * E;
        ag.env_step_dev = c->la_steps + i;
    }
    c->la_obs = ob;
    return GALA_OK;
}

// One iteration of the closed loop without the gossip step, enqueued on the agent's stream: the observation the
// rollout starts from, T x (act, environment step), the learner step, and the advance of the step counter.
static int actor_iteration(gala_ctx* c, int agent, unsigned long long env_seed) {
    Agent& ag = c->agents[agent];
    const int T = c->T, E = c->E;
    const long obs_elems = c->conv ? kFramePix : c->obs_dim;
    const long obs_bytes = obs_elems * (c->conv ? 1 : 4);
    uint8_t* obs = reinterpret_cast<uint8_t*>(ag.loop_obs);
    EnvArgs ea{};
    ea.seed = env_seed; ea.agent = agent; ea.n_actions = c->A; ea.step_base = ag.env_step_dev;
    ea.uniforms = ag.loop_uniforms; ea.obs_elems = obs_elems; ea.frames = c->conv ? 1 : 0;
    EnvArgs first = ea;   // the environment is a function of the step: the first observation is produced again
    first.obs_step = 0; first.obs_out = obs;
    LAUNCH(T_ENV, ag.stream, launch_env(first, E, ag.stream));
    for (int t = 0; t < T; t++) {
        int r = gala_act(c, agent, obs + (long)t * E * obs_bytes, ag.loop_uniforms, ag.loop_actions + (long)t * E, nullptr);
        if (r != GALA_OK) return r;
        EnvArgs st = ea;
        st.step = t; st.actions = ag.loop_actions + (long)t * E;
        st.rewards = ag.loop_rewards + (long)t * E; st.dones = ag.loop_dones + (long)t * E;
        st.obs_step = t + 1; st.obs_out = obs + (long)(t + 1) * E * obs_bytes;
        LAUNCH(T_ENV, ag.stream, launch_env(st, E, ag.stream));
    }
    gala_rollout ro{obs, ag.loop_actions, ag.loop_rewards, ag.loop_dones};
    c->cur_ctas = c->agent_ctas;
    int r = learn_range(c, agent, 1, &ro, ag.stream);
    c->cur_ctas = 0;
    if (r != GALA_OK) return r;
    LAUNCH(T_ENV, ag.stream, launch_env_advance(ag.env_step_dev, T, ag.stream));
    return GALA_OK;
}

int gala_actor_loop(gala_ctx* c, int agent, int iterations, unsigned long long env_seed) {
    if (!valid_agent(c, agent) || iterations < 0) return fail(c, GALA_EINVAL, "gala_actor_loop: bad agent or iteration count");
    if (c->topo.kind == GALA_TOPO_COMPLETE)
        return fail(c, GALA_ESTATE, "gala_actor_loop: the complete graph (gradient all-reduce) exists only as gala_step_sync");
    Agent& ag = c->agents[agent];
    const int T = c->T;
    { int r0 = ensure_loop_buffers(c); if (r0 != GALA_OK) return r0; }
    if (ag.loop_seed != env_seed) {   // the captured iteration carries the seed
        if (ag.loop_graph.exec) { cudaGraphExecDestroy(ag.loop_graph.exec); ag.loop_graph.exec = nullptr; }
        ag.loop_graph.failed = false;
        ag.loop_seed = env_seed; ag.loop_seen = 0;
    }
    const unsigned long long outside = (1ull << T_SWEEP_SYNC) | (1ull << T_SWEEP_AGENT);
    {
        int r0 = own_stream_begin(c, ag);
        if (r0 != GALA_OK) return r0;
    }
    for (int it = 0; it < iterations; it++) {
        if (ag.pending) {  // a gradient that no gossip step has consumed: apply it without mixing, publish
            int r0 = sweep_agent(c, agent, false);
            if (r0 != GALA_OK) return r0;
            ag.round++;
        }
        StepGraph& g = ag.loop_graph;
        const bool graphs = c->use_graphs >= 1 && (c->profile_mask & ~outside) == 0 && !c->legacy_conv && !g.failed;
        int r = GALA_OK;
        if (graphs && g.exec) {            // third iteration on: one graph launch
            CK(cudaGraphLaunch(g.exec, ag.stream));
            c->launches += g.launches;
            for (int k = 0; k < T_COUNT; k++) c->tag_launches[k] += g.tag_launches[k];
            ag.pending = true; ag.frames += c->S;
        } else if (graphs && ag.loop_seen >= 1 && cudaStreamBeginCapture(ag.stream, cudaStreamCaptureModeRelaxed) == cudaSuccess) {
            const long long l0 = c->launches;   // second iteration: captured, instantiated, launched
            long long t0[T_COUNT];
            for (int k = 0; k < T_COUNT; k++) t0[k] = c->tag_launches[k];
            r = actor_iteration(c, agent, env_seed);
            cudaGraph_t graph = nullptr;
            cudaError_t e = cudaStreamEndCapture(ag.stream, &graph);
            if (r == GALA_OK && e == cudaSuccess && graph) e = cudaGraphInstantiate(&g.exec, graph, 0);
            if (graph) cudaGraphDestroy(graph);
            if (r != GALA_OK || e != cudaSuccess || !g.exec) {
                (void)cudaGetLastError();
                g.failed = true; g.exec = nullptr;
                c->launches = l0;
                for (int k = 0; k < T_COUNT; k++) c->tag_launches[k] = t0[k];
                if (r != GALA_OK) return r;
                ag.frames -= c->S;     // counted again by the direct pass
                if ((r = actor_iteration(c, agent, env_seed)) != GALA_OK) return r;
            } else {
                g.launches = c->launches - l0;
                for (int k = 0; k < T_COUNT; k++) g.tag_launches[k] = c->tag_launches[k] - t0[k];
                CK(cudaGraphLaunch(g.exec, ag.stream));
            }
        } else {                           // first iteration (or no graphs): direct launches
            (void)cudaGetLastError();
            if ((r = actor_iteration(c, agent, env_seed)) != GALA_OK) return r;
        }
        ag.loop_seen++;
        ag.env_step += T;
        if ((r = gala_gossip(c, agent)) != GALA_OK) return r;
    }
    return GALA_OK;
}

static int main_stream_joins_agents(gala_ctx* c);
static int agents_join_main_stream(gala_ctx* c);
static int sync_round_body(gala_ctx* c, const gala_rollout* ros);

// The acting part of a lockstep iteration on the main stream: first observations, T x (forward of all agents,
// draw + environment step of all agents), step counters advanced.
static int act_all(gala_ctx* c, unsigned long long env_seed) {
    const int T = c->T, E = c->E, n = c->n;
    const long obs_elems = c->conv ? kFramePix : c->obs_dim;
    const long obs_bytes = obs_elems * (c->conv ? 1 : 4);
    const long per_obs = (long)(T + 1) * E * obs_bytes;
    cudaStream_t st = c->main_stream;
    EnvActArgs ea{};
    ea.seed = env_seed; ea.n_actions = c->A; ea.frames = c->conv ? 1 : 0; ea.step_base = c->la_steps;
    ea.logits = c->logits; ea.logits_stride = c->B * c->A;
    ea.actions = c->la_actions; ea.rewards = c->la_rewards; ea.dones = c->la_dones; ea.te_stride = (long)T * E;
    ea.obs_out = c->la_obs; ea.obs_agent_stride = per_obs; ea.obs_elems = obs_elems;
    EnvActArgs first = ea;   // the environment is a function of the step: the first observation is produced again
    first.draw = 0; first.step = 0; first.obs_off = 0;
    LAUNCH(T_ENV, st, launch_env_act_all(first, E, n, st));
    for (int t = 0; t < T; t++) {
        for (int a0 = 0; a0 < n; a0 += kBatch) {
            const int cnt = n - a0 < kBatch ? n - a0 : kBatch;
            PtrBatch pb{};
            for (int i = 0; i < cnt; i++) pb.p[i] = c->la_obs + (long)(a0 + i) * per_obs + (long)t * E * obs_bytes;
            // conv net: the trunk up to the (possibly split) hidden-layer product; the kernel that draws the actions
            // finishes the hidden layer and forms the policy head of its environment itself
            HiddenPending pend;
            int r = forward(c, a0, cnt, pb, E, st, nullptr, c->conv ? &pend : nullptr);
            if (r != GALA_OK) return r;
            EnvActArgs sa = ea;
            sa.agent0 = a0;
            sa.draw = 1; sa.step = t; sa.te_off = (long)t * E; sa.obs_off = (long)(t + 1) * E * obs_bytes;
            if (c->conv) {
                sa.H = kHidden; sa.split = pend.split;
                sa.partials = c->splitk_ws + (long)a0 * c->splitk_group_stride;
                sa.split_stride = pend.count; sa.partial_group_stride = c->splitk_group_stride;
                sa.hid = c->hid; sa.h_stride = c->B * kHidden;
                sa.params = c->x; sa.p_stride = c->d_pad;
                sa.piw = c->cl.piw; sa.pib = c->cl.pib; sa.fcb = c->cl.fcb;
            }
            LAUNCH(T_ENV, st, launch_env_act_all(sa, E, cnt, st));
        }
    }
    LAUNCH(T_ENV, st, launch_env_advance_all(c->la_steps, n, T, st));
    return GALA_OK;
}

int gala_actor_loop_all(gala_ctx* c, int iterations, unsigned long long env_seed) {
    if (!c || iterations < 0) return c ? fail(c, GALA_EINVAL, "gala_actor_loop_all: negative iteration count") : GALA_EINVAL;
    if (c->legacy_conv) return fail(c, GALA_ESTATE, "gala_actor_loop_all: not with the earlier convolution kernels");
    const int n = c->n, T = c->T;
    { int r0 = ensure_loop_buffers(c); if (r0 != GALA_OK) return r0; }
    if (c->la_seed != env_seed) {   // the captured part carries the seed
        if (c->la_graph.exec) { cudaGraphExecDestroy(c->la_graph.exec); c->la_graph.exec = nullptr; }
        c->la_graph.failed = false;
        c->la_seed = env_seed; c->la_seen = 0;
    }
    std::vector<gala_rollout> ros((size_t)n);
    for (int i = 0; i < n; i++) {
        Agent& ag = c->agents[i];
        ros[i] = gala_rollout{ag.loop_obs, ag.loop_actions, ag.loop_rewards, ag.loop_dones};
    }
    cudaStream_t st = c->main_stream;
    const unsigned long long outside = (1ull << T_SWEEP_SYNC) | (1ull << T_SWEEP_AGENT);
    // the whole loop runs on the main stream: ordered against the agents' streams once on either side
    if (iterations > 0) { int r0 = main_stream_joins_agents(c); if (r0 != GALA_OK) return r0; }
    for (int it = 0; it < iterations; it++) {
        StepGraph& g = c->la_graph;
        const bool graphs = c->use_graphs >= 1 && (c->profile_mask & ~outside) == 0 && !g.failed;
        int r = GALA_OK;
        if (graphs && g.exec) {            // third iteration on: one graph launch
            CK(cudaGraphLaunch(g.exec, st));
            c->launches += g.launches;
            for (int k = 0; k < T_COUNT; k++) c->tag_launches[k] += g.tag_launches[k];
        } else if (graphs && c->la_seen >= 1 && cudaStreamBeginCapture(st, cudaStreamCaptureModeRelaxed) == cudaSuccess) {
            const long long l0 = c->launches;   // second iteration: captured, instantiated, launched
            long long t0[T_COUNT];
            for (int k = 0; k < T_COUNT; k++) t0[k] = c->tag_launches[k];
            r = act_all(c, env_seed);
            cudaGraph_t graph = nullptr;
            cudaError_t e = cudaStreamEndCapture(st, &graph);
            if (r == GALA_OK && e == cudaSuccess && graph) e = cudaGraphInstantiate(&g.exec, graph, 0);
            if (graph) cudaGraphDestroy(graph);
            if (r != GALA_OK || e != cudaSuccess || !g.exec) {
                (void)cudaGetLastError();
                g.failed = true; g.exec = nullptr;
                c->launches = l0;
                for (int k = 0; k < T_COUNT; k++) c->tag_launches[k] = t0[k];
                if (r != GALA_OK) return r;
                if ((r = act_all(c, env_seed)) != GALA_OK) return r;
            } else {
                g.launches = c->launches - l0;
                for (int k = 0; k < T_COUNT; k++) g.tag_launches[k] = c->tag_launches[k] - t0[k];
                CK(cudaGraphLaunch(g.exec, st));
            }
        } else {                           // first iteration (or no graphs): direct launches
            (void)cudaGetLastError();
            if ((r = act_all(c, env_seed)) != GALA_OK) return r;
        }
        c->la_seen++;
        for (int i = 0; i < n; i++) c->agents[i].env_step += T;
        if ((r = sync_round_body(c, ros.data())) != GALA_OK) { (void)agents_join_main_stream(c); return r; }
    }
    return iterations > 0 ? agents_join_main_stream(c) : GALA_OK;
}

int gala_actor_read(gala_ctx* c, int agent, void* obs, int* actions, float* rewards, unsigned char* dones,
                    long long* next_step) {
    if (!valid_agent(c, agent)) return fail(c, GALA_EINVAL, "gala_actor_read: bad agent");
    Agent& ag = c->agents[agent];
    if (!ag.loop_obs) return fail(c, GALA_ESTATE, "gala_actor_read: gala_actor_loop has not run for this agent");
    { int r = settle_agent(c, agent); if (r != GALA_OK) return r; }
    const long obs_bytes = (c->conv ? kFramePix : (long)c->obs_dim * 4);
    const size_t TE = (size_t)c->T * c->E;
    if (obs) CK(cudaMemcpy(obs, ag.loop_obs, (size_t)(c->T + 1) * c->E * obs_bytes, cudaMemcpyDeviceToHost));
    if (actions) CK(cudaMemcpy(actions, ag.loop_actions, TE * sizeof(int), cudaMemcpyDeviceToHost));
    if (rewards) CK(cudaMemcpy(rewards, ag.loop_rewards, TE * sizeof(float), cudaMemcpyDeviceToHost));
    if (dones) CK(cudaMemcpy(dones, ag.loop_dones, TE, cudaMemcpyDeviceToHost));
    if (next_step) *next_step = ag.env_step;
    return GALA_OK;
}

int gala_learn(gala_ctx* c, int agent, const gala_rollout* ro) {
    if (!valid_agent(c, agent) || !ro || !ro->obs || !ro->actions || !ro->rewards || !ro->dones)
        return fail(c, GALA_EINVAL, "gala_learn: bad agent or null rollout pointer");
    Agent& ag = c->agents[agent];
    if (ag.pending) {  // apply the earlier gradient without mixing, publish
        int r = sweep_agent(c, agent, false);
        if (r != GALA_OK) return r;
        ag.round++;
    }
    int r = own_stream_begin(c, ag);
    if (r != GALA_OK) return r;
    c->cur_ctas = c->agent_ctas;
    r = learn_range_cached(c, agent, 1, ro, ag.stream);
    c->cur_ctas = 0;
    return r;
}

int gala_gossip(gala_ctx* c, int agent) {
    if (!valid_agent(c, agent)) return fail(c, GALA_EINVAL, "gala_gossip: bad agent");
    if (c->topo.kind == GALA_TOPO_COMPLETE)
        return fail(c, GALA_ESTATE, "gala_gossip: the complete graph (gradient all-reduce) exists only as gala_step_sync");
    int r = sweep_agent(c, agent, true);
    if (r != GALA_OK) return r;
    c->agents[agent].round++;
    return GALA_OK;
}

// A list of distinct, valid agents.
static int check_agent_list(gala_ctx* c, const int* agents, int m, const char* who) {
    if (!c) return GALA_EINVAL;
    if (!agents || m < 0 || m > c->n) return fail(c, GALA_EINVAL, "%s: null list or more entries than agents", who);
    bool seen[256] = {};
    for (int k = 0; k < m; k++) {
        if (!valid_agent(c, agents[k])) return fail(c, GALA_EINVAL, "%s: entry %d is not an agent", who, k);
        if (seen[agents[k]]) return fail(c, GALA_EINVAL, "%s: agent %d is listed twice", who, agents[k]);
        seen[agents[k]] = true;
    }
    return GALA_OK;
}

int gala_learn_many(gala_ctx* c, const int* agents, const gala_rollout* ros, int m) {
    int r = check_agent_list(c, agents, m, "gala_learn_many");
    if (r != GALA_OK) return r;
    if (m == 0) return GALA_OK;
    if (!ros) return fail(c, GALA_EINVAL, "gala_learn_many: null rollouts");
    for (int k = 0; k < m; k++)
        if (!ros[k].obs || !ros[k].actions || !ros[k].rewards || !ros[k].dones)
            return fail(c, GALA_EINVAL, "gala_learn_many: null rollout pointer in entry %d", k);
    // the grouped kernels are those of the conv net with the fused heads; everything else goes agent by agent
    if (!c->conv || !c->fused_heads || c->legacy_conv) {
        for (int k = 0; k < m; k++)
            if ((r = gala_learn(c, agents[k], &ros[k])) != GALA_OK) return r;
        return GALA_OK;
    }
    const int lane = c->next_lane;
    c->next_lane = (c->next_lane + 1) % c->n_lanes;
    gala_ctx::Lane& L = c->glane[lane];
    if ((r = lane_acquire(c, lane, agents, m)) != GALA_OK) return r;
    // gradients that no gossip step has consumed are applied without mixing and published first
    std::vector<int> pend;
    for (int k = 0; k < m; k++)
        if (c->agents[agents[k]].pending) pend.push_back(agents[k]);
    if (!pend.empty()) {
        if ((r = sweep_group(c, lane, pend.data(), (int)pend.size(), false)) != GALA_OK) return r;
        for (int i : pend) c->agents[i].round++;
    }
    // several kernel classes timed at once: one stream, so that an event pair brackets a kernel
    const unsigned long long outside = (1ull << T_SWEEP_SYNC) | (1ull << T_SWEEP_AGENT) | (1ull << T_SAMPLE);
    const unsigned long long inside = c->profile_mask & ~outside;
    cudaStream_t side = (inside & (inside - 1)) != 0 ? nullptr : L.side;
    c->cur_fork = L.fork; c->cur_join = L.join;
    for (int k0 = 0; k0 < m && r == GALA_OK; k0 += kBatch) {
        const int cnt = m - k0 < kBatch ? m - k0 : kBatch;
        AgentMap am{};
        am.on = 1;
        for (int e = 0; e < cnt; e++) am.v[e] = (unsigned char)agents[k0 + e];
        c->cur_map = &am;
        r = learn_range(c, 0, cnt, ros + k0, L.st, side);
        c->cur_map = nullptr;
    }
    c->cur_fork = c->ev_fork; c->cur_join = c->ev_join;
    const int r2 = lane_release(c, lane, agents, m);
    return r != GALA_OK ? r : r2;
}

int gala_gossip_many(gala_ctx* c, const int* agents, int m) {
    int r = check_agent_list(c, agents, m, "gala_gossip_many");
    if (r != GALA_OK) return r;
    if (m == 0) return GALA_OK;
    if (c->topo.kind == GALA_TOPO_COMPLETE)
        return fail(c, GALA_ESTATE, "gala_gossip_many: the complete graph (gradient all-reduce) exists only as gala_step_sync");
    // the lane of the learner steps these agents' gradients come from, so that nothing waits across lanes
    const int last = c->agents[agents[0]].group_lane;
    const int lane = last >= 0 ? last : c->next_lane;
    if ((r = lane_acquire(c, lane, agents, m)) != GALA_OK) return r;
    if ((r = sweep_group(c, lane, agents, m, true)) != GALA_OK) return r;
    for (int k = 0; k < m; k++) c->agents[agents[k]].round++;
    return lane_release(c, lane, agents, m);
}

int gala_poll_agent(gala_ctx* c, int agent, int* busy) {
    if (!valid_agent(c, agent) || !busy) return fail(c, GALA_EINVAL, "gala_poll_agent: bad agent or null output");
    Agent& ag = c->agents[agent];
    *busy = 0;
    cudaError_t e = ag.version > 0 ? cudaEventQuery(ag.pub_event[ag.version % kSnapSlots]) : cudaSuccess;
    if (e == cudaSuccess && (ag.pending || ag.dirty)) {   // work after the last optimiser step: ask the streams
        if (ag.group_lane >= 0) e = cudaStreamQuery(c->glane[ag.group_lane].st);
        if (e == cudaSuccess) e = cudaStreamQuery(ag.stream);
    }
    if (e == cudaErrorNotReady) { *busy = 1; return GALA_OK; }
    if (e != cudaSuccess) return fail(c, GALA_ECUDA, "gala_poll_agent: %s", cudaGetErrorString(e));
    return GALA_OK;
}

int gala_delay(gala_ctx* c, int agent, int usec) {
    if (!valid_agent(c, agent) || usec < 0 || usec > 100000)
        return fail(c, GALA_EINVAL, "gala_delay: bad agent or delay outside 0..100000 us");
    if (usec == 0) return GALA_OK;
    Agent& ag = c->agents[agent];
    int r = own_stream_begin(c, ag);
    if (r != GALA_OK) return r;
    CK(launch_delay((unsigned long long)usec, ag.stream));
    return GALA_OK;
}

// The main stream waits for everything the agents have enqueued, also on the lanes of the grouped calls.
static int main_stream_joins_agents(gala_ctx* c) {
    cudaStream_t st = c->main_stream;
    for (int i = 0; i < c->n; i++) {
        Agent& ag = c->agents[i];
        if (ag.group_lane >= 0) {
            CK(cudaStreamWaitEvent(st, c->glane[ag.group_lane].done, 0));
            ag.group_lane = -1;
        }
        CK(cudaEventRecord(ag.fence, ag.stream));
        CK(cudaStreamWaitEvent(st, ag.fence, 0));
    }
    return GALA_OK;
}
// The agents' streams wait for what the main stream holds now.
static int agents_join_main_stream(gala_ctx* c) {
    CK(cudaEventRecord(c->main_event, c->main_stream));
    for (int i = 0; i < c->n; i++) {
        CK(cudaStreamWaitEvent(c->agents[i].stream, c->main_event, 0));
        c->agents[i].dirty = true;     // a grouped call must be ordered behind this round through the agent's stream
    }
    return GALA_OK;
}

// One synchronous round on the main stream, without the ordering against the agents' streams on either side.
static int sync_round_body(gala_ctx* c, const gala_rollout* ros) {
    const int n = c->n;
    cudaStream_t st = c->main_stream;
    if (ros) {
        // Timing several kernel classes of the step at once: one stream, so that an event pair brackets a kernel
        // and not its wait for the SMs that the other stream's kernels hold.
        const unsigned long long outside = (1ull << T_SWEEP_SYNC) | (1ull << T_SWEEP_AGENT) | (1ull << T_SAMPLE);
        const unsigned long long inside = c->profile_mask & ~outside;
        cudaStream_t side = (inside & (inside - 1)) != 0 ? nullptr : c->side_stream;
        for (int a0 = 0; a0 < n; a0 += kBatch) {
            const int cnt = n - a0 < kBatch ? n - a0 : kBatch;
            int r = learn_range_cached(c, a0, cnt, ros + a0, st, side);
            if (r != GALA_OK) return r;
        }
    }
    int off[2] = {0, 0};
    int np = topo_offsets(c->topo, n, c->sync_round, off);
    if (c->topo.kind == GALA_TOPO_COMPLETE) {
        // synchronous A2C baseline: average the gradients over all agents, clip the average, and let every
        // agent take the same RMSProp step; no parameter mixing
        np = 0;
        LAUNCH(T_GRAD_NORM, st, launch_allreduce_grads(c->g, n, c->d_pad, st));
        LAUNCH(T_GRAD_NORM, st, launch_grad_norm(c->g, c->d, c->d_pad, 0, n, c->hp.max_grad_norm, c->norm_partial,
                                                 c->norm_ticket, c->norm, c->clip, st));
    }
    SweepHp hp{c->hp.lr, c->hp.rms_alpha, c->hp.rms_eps};
    if (c->track_updates) {   // the norm of the step this pass is about to take, from the same g, clip and v
        LAUNCH(T_GRAD_NORM, st, launch_update_norm(c->g, c->v, c->clip, n, c->d_pad, hp, c->upd_partial, c->upd_ticket,
                                                   c->upd_out, st));
        c->upd_valid = true;
    }
    LAUNCH(T_SWEEP_SYNC, st, launch_sweep_sync(c->x, c->g, c->v, c->clip, c->conv ? c->shadow : nullptr, n, c->d_pad, np, off, hp,
                                            c->error_word, st));
    for (int i = 0; i < n; i++) {
        c->agents[i].pending = false;
        c->agents[i].round++;
    }
    c->sync_round++;
    return GALA_OK;
}

int gala_step_sync(gala_ctx* c, const gala_rollout* ros) {
    if (!c) return GALA_EINVAL;
    if (ros)
        for (int i = 0; i < c->n; i++)
            if (!ros[i].obs || !ros[i].actions || !ros[i].rewards || !ros[i].dones)
                return fail(c, GALA_EINVAL, "gala_step_sync: null rollout pointer for agent %d", i);
    int r = main_stream_joins_agents(c);
    if (r != GALA_OK) return r;
    if ((r = sync_round_body(c, ros)) != GALA_OK) return r;
    return agents_join_main_stream(c);
}

int gala_sync_agent(gala_ctx* c, int agent, int timeout_ms) {
    if (!valid_agent(c, agent)) return fail(c, GALA_EINVAL, "gala_sync_agent: bad agent");
    Agent& ag = c->agents[agent];
    int r = ag.group_lane >= 0 ? host_wait(c, c->glane[ag.group_lane].st, timeout_ms) : GALA_OK;
    if (r != GALA_OK) return r;
    if ((r = host_wait(c, ag.stream, timeout_ms)) != GALA_OK) return r;
    return check_error_word(c);
}

int gala_sync_all(gala_ctx* c, int timeout_ms) {
    if (!c) return GALA_EINVAL;
    int r = host_wait(c, c->main_stream, timeout_ms);
    if (r != GALA_OK) return r;
    for (gala_ctx::Lane& L : c->glane)
        if ((r = host_wait(c, L.st, timeout_ms)) != GALA_OK) return r;
    for (int i = 0; i < c->n; i++)
        if ((r = host_wait(c, c->agents[i].stream, timeout_ms)) != GALA_OK) return r;
    return check_error_word(c);
}

int gala_in_peers(const gala_ctx* c, long long round, int agent, int* peers, int* n) {
    if (!valid_agent(c, agent) || !peers || !n || round < 0 || c->topo.kind == GALA_TOPO_COMPLETE) return GALA_EINVAL;
    int off[2];
    const int np = topo_offsets(c->topo, c->n, round, off);
    for (int j = 0; j < np; j++) peers[j] = ((agent - off[j]) % c->n + c->n) % c->n;
    *n = np;
    return GALA_OK;
}

int gala_get_state(gala_ctx* c, int agent, float* params, float* sq_avg, float* grad, long long* round) {
    if (!valid_agent(c, agent)) return fail(c, GALA_EINVAL, "gala_get_state: bad agent");
    { int r = settle_agent(c, agent); if (r != GALA_OK) return r; }
    const size_t bytes = (size_t)c->d * sizeof(float);
    if (params) CK(cudaMemcpy(params, c->x + (long)agent * c->d_pad, bytes, cudaMemcpyDefault));
    if (sq_avg) CK(cudaMemcpy(sq_avg, c->v + (long)agent * c->d_pad, bytes, cudaMemcpyDefault));
    if (grad) CK(cudaMemcpy(grad, c->g + (long)agent * c->d_pad, bytes, cudaMemcpyDefault));
    if (round) *round = c->agents[agent].round;
    return check_error_word(c);
}

int gala_set_state(gala_ctx* c, int agent, const float* params, const float* sq_avg, long long round) {
    if (!valid_agent(c, agent) || round < 0) return fail(c, GALA_EINVAL, "gala_set_state: bad agent or round");
    Agent& ag = c->agents[agent];
    { int r = settle_agent(c, agent); if (r != GALA_OK) return r; }
    const size_t bytes = (size_t)c->d * sizeof(float);
    if (params) {
        int r = copy_in(c, c->x + (long)agent * c->d_pad, params, bytes, ag.stream);
        if (r != GALA_OK) return r;
        if (c->conv) {
            LAUNCH(T_CAST, ag.stream, launch_cast_bf16(c->x + (long)agent * c->d_pad, c->shadow + (long)agent * c->d_pad, c->d_pad, ag.stream));
            CK(cudaStreamSynchronize(ag.stream));
        }
    }
    if (sq_avg) {
        int r = copy_in(c, c->v + (long)agent * c->d_pad, sq_avg, bytes, ag.stream);
        if (r != GALA_OK) return r;
    }
    ag.round = round;
    if (agent == 0) c->sync_round = round;
    return GALA_OK;
}

int gala_set_grad(gala_ctx* c, int agent, const float* grad, float clip_coef) {
    if (!valid_agent(c, agent) || !grad) return fail(c, GALA_EINVAL, "gala_set_grad: bad agent or null gradient");
    Agent& ag = c->agents[agent];
    int r = settle_agent(c, agent);
    if (r != GALA_OK) return r;
    r = copy_in(c, c->g + (long)agent * c->d_pad, grad, (size_t)c->d * sizeof(float), ag.stream);
    if (r != GALA_OK) return r;
    if (clip_coef >= 0.0f) {
        if ((r = copy_in(c, c->clip + agent, &clip_coef, sizeof(float), ag.stream)) != GALA_OK) return r;
    } else {
        LAUNCH(T_GRAD_NORM, ag.stream, launch_grad_norm(c->g, c->d, c->d_pad, agent, 1, c->hp.max_grad_norm, c->norm_partial, c->norm_ticket,
                                c->norm, c->clip, ag.stream));
        CK(cudaStreamSynchronize(ag.stream));
    }
    ag.pending = true;
    return GALA_OK;
}

int gala_consensus_distance(gala_ctx* c, double* out) {
    if (!c || !out) return GALA_EINVAL;
    int r = gala_sync_all(c, -1);
    if (r != GALA_OK) return r;
    LAUNCH(T_GRAD_NORM, c->main_stream, launch_consensus(c->x, c->n, c->d, c->d_pad, c->cons_partial, c->cons_ticket,
                                                        c->cons_out, c->main_stream));
    CK(cudaStreamSynchronize(c->main_stream));
    double sq = 0.0;
    CK(cudaMemcpy(&sq, c->cons_out, sizeof sq, cudaMemcpyDeviceToHost));
    *out = std::sqrt(sq);
    return GALA_OK;
}

int gala_track_updates(gala_ctx* c, int on) {
    if (!c) return GALA_EINVAL;
    c->track_updates = on != 0;
    if (!on) c->upd_valid = false;
    return GALA_OK;
}

int gala_update_norm(gala_ctx* c, double* out) {
    if (!c || !out) return GALA_EINVAL;
    if (!c->upd_valid) return fail(c, GALA_EINVAL, "gala_update_norm: no synchronous round since gala_track_updates(ctx, 1)");
    int r = host_wait(c, c->main_stream, -1);
    if (r != GALA_OK) return r;
    double sq = 0.0;
    CK(cudaMemcpy(&sq, c->upd_out, sizeof sq, cudaMemcpyDeviceToHost));
    *out = std::sqrt(sq);
    return GALA_OK;
}

int gala_set_graphs(gala_ctx* c, int on) {
    if (!c) return GALA_EINVAL;
    if (on < 0 || on > 2) return fail(c, GALA_EINVAL, "gala_set_graphs: mode must be 0, 1 or 2");
    c->use_graphs = on;
    return GALA_OK;
}

int gala_debug_wait_runs_out(gala_ctx* c, int agent, int polls) {
    if (!valid_agent(c, agent) || polls < 1 || polls > 100000)
        return fail(c, GALA_EINVAL, "gala_debug_wait_runs_out: bad agent or poll count outside 1..100000");
    Agent& ag = c->agents[agent];
    int r = own_stream_begin(c, ag);
    if (r != GALA_OK) return r;
    CK(launch_wait_runs_out((unsigned)polls, c->error_word, ag.stream));
    return GALA_OK;
}

int gala_set_group_lanes(gala_ctx* c, int lanes) {
    if (!c || lanes < 1 || lanes > 2) return fail(c, GALA_EINVAL, "gala_set_group_lanes: 1 or 2");
    c->n_lanes = lanes;
    c->next_lane = 0;
    return GALA_OK;
}

int gala_set_agent_ctas(gala_ctx* c, int ctas) {
    if (!c || ctas < 0) return fail(c, GALA_EINVAL, "gala_set_agent_ctas: negative budget");
    c->agent_ctas = ctas >= sm_count() ? 0 : ctas;
    return GALA_OK;
}

int gala_set_stale_timeout(gala_ctx* c, int timeout_ms) {
    if (!c || timeout_ms < 0) return GALA_EINVAL;
    c->stale_timeout_ms = timeout_ms;
    return GALA_OK;
}

int gala_param_count(const gala_ctx* c, long long* d, long long* d_padded) {
    if (!c) return GALA_EINVAL;
    if (d) *d = c->d;
    if (d_padded) *d_padded = c->d_pad;
    return GALA_OK;
}

int gala_losses(gala_ctx* c, int agent, float out[4]) {
    if (!valid_agent(c, agent) || !out) return fail(c, GALA_EINVAL, "gala_losses: bad argument");
    { int r = settle_agent(c, agent); if (r != GALA_OK) return r; }
    CK(cudaMemcpy(out, c->losses + (long)agent * 4, 3 * sizeof(float), cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(out + 3, c->norm + agent, sizeof(float), cudaMemcpyDeviceToHost));
    return GALA_OK;
}

int gala_losses_all(gala_ctx* c, float* out) {
    if (!c || !out) return fail(c, GALA_EINVAL, "gala_losses_all: bad argument");
    CK(cudaStreamSynchronize(c->main_stream));
    for (gala_ctx::Lane& L : c->glane) CK(cudaStreamSynchronize(L.st));
    for (Agent& a : c->agents) CK(cudaStreamSynchronize(a.stream));
    std::vector<float> nrm(c->n);
    CK(cudaMemcpy(out, c->losses, (size_t)c->n * 4 * sizeof(float), cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(nrm.data(), c->norm, (size_t)c->n * sizeof(float), cudaMemcpyDeviceToHost));
    for (int i = 0; i < c->n; i++) out[4 * i + 3] = nrm[i];
    return GALA_OK;
}

int gala_stats(gala_ctx* c, int agent, long long out[8]) {
    if (!valid_agent(c, agent) || !out) return GALA_EINVAL;
    const Agent& a = c->agents[agent];
    out[0] = a.frames; out[1] = a.round; out[2] = a.mixes; out[3] = a.skipped;
    out[4] = a.stale_sum; out[5] = a.stale_max; out[6] = a.version; out[7] = a.stale_waits;
    return GALA_OK;
}

int gala_last_mix(gala_ctx* c, int agent, int* peers, long long* versions, int* n, int* mixed) {
    if (!valid_agent(c, agent)) return GALA_EINVAL;
    const Agent& a = c->agents[agent];
    for (int j = 0; j < a.last_n; j++) {
        if (peers) peers[j] = a.last_peers[j];
        if (versions) versions[j] = a.last_versions[j];
    }
    if (n) *n = a.last_n;
    if (mixed) *mixed = a.last_mixed;
    return GALA_OK;
}

int gala_get_snapshot(gala_ctx* c, int agent, long long version, float* out) {
    if (!valid_agent(c, agent) || !out) return fail(c, GALA_EINVAL, "gala_get_snapshot: bad argument");
    Agent& a = c->agents[agent];
    if (version < 1 || version > a.version || version < a.version - 1)
        return fail(c, GALA_ESTATE, "snapshot version %lld of agent %d is not held (newest %lld)", version, agent,
                    a.version);
    { int r = settle_agent(c, agent); if (r != GALA_OK) return r; }
    CK(cudaMemcpy(out, c->snap + ((long)agent * kSnapSlots + version % kSnapSlots) * c->d_pad, (size_t)c->d * sizeof(float),
                  cudaMemcpyDefault));
    return GALA_OK;
}

int gala_set_stream(gala_ctx* c, int agent, void* cuda_stream) {
    if (!valid_agent(c, agent)) return GALA_EINVAL;
    Agent& a = c->agents[agent];
    { int r = settle_agent(c, agent); if (r != GALA_OK) return r; }
    a.stream = cuda_stream ? reinterpret_cast<cudaStream_t>(cuda_stream) : a.lib_stream;
    return GALA_OK;
}

int gala_debug_read(gala_ctx* c, int agent, int what, float* out, long long count) {
    if (!valid_agent(c, agent) || !out || count < 0) return fail(c, GALA_EINVAL, "gala_debug_read: bad argument");
    { int r = settle_agent(c, agent); if (r != GALA_OK) return r; }
    const long B = c->B, S = c->S;
    const int A = c->A;
    const float* src = nullptr;
    long avail = 0;
    switch (what) {
        case 0: src = c->logits + (long)agent * B * A; avail = B * A; break;
        case 1: src = c->values + (long)agent * B; avail = B; break;
        case 2: src = c->returns + (long)agent * S; avail = S; break;
        case 3: src = c->adv + (long)agent * S; avail = S; break;
        case 4: src = c->dlogits + (long)agent * S * A; avail = S * A; break;
        case 5: src = c->dvalues + (long)agent * S; avail = S; break;
        default: break;
    }
    if (src) {
        if (count > avail) return fail(c, GALA_EINVAL, "gala_debug_read: count %lld > %ld", count, avail);
        CK(cudaMemcpy(out, src, (size_t)count * sizeof(float), cudaMemcpyDefault));
        return GALA_OK;
    }
    if (what == 20) {   // the bf16 copy of the parameters that the trunk products read
        if (!c->conv) return fail(c, GALA_EINVAL, "gala_debug_read: no bf16 parameter copy for this network");
        if (count > c->d) return fail(c, GALA_EINVAL, "gala_debug_read: count %lld > %ld", count, c->d);
        std::vector<__nv_bfloat16> tmp((size_t)count);
        CK(cudaMemcpy(tmp.data(), c->shadow + (long)agent * c->d_pad, (size_t)count * 2, cudaMemcpyDeviceToHost));
        std::vector<float> f((size_t)count);
        for (long long i = 0; i < count; i++) f[i] = __bfloat162float(tmp[i]);
        CK(cudaMemcpy(out, f.data(), (size_t)count * sizeof(float), cudaMemcpyDefault));
        return GALA_OK;
    }
    if (what >= 10 && what <= 13) {
        const int l = what - 10;
        const void* p = nullptr;
        bool bf = false;
        if (c->conv) {
            const int P[3] = {400, 81, 49};
            bf = true;
            if (l < 3) { p = c->act[l] + (long)agent * B * P[l] * kConvCout[l]; avail = B * P[l] * kConvCout[l]; }
            else { p = c->hid + (long)agent * B * kHidden; avail = B * kHidden; }
        } else {
            if (l == 0) p = c->h1 + (long)agent * B * c->H;
            else if (l == 1) p = c->h2 + (long)agent * B * c->H;
            avail = B * c->H;
        }
        if (!p) return fail(c, GALA_EINVAL, "gala_debug_read: no such layer");
        if (count > avail) return fail(c, GALA_EINVAL, "gala_debug_read: count %lld > %ld", count, avail);
        if (!bf) {
            CK(cudaMemcpy(out, p, (size_t)count * sizeof(float), cudaMemcpyDefault));
            return GALA_OK;
        }
        std::vector<__nv_bfloat16> tmp((size_t)count);
        CK(cudaMemcpy(tmp.data(), p, (size_t)count * 2, cudaMemcpyDeviceToHost));
        std::vector<float> f((size_t)count);
        for (long long i = 0; i < count; i++) f[i] = __bfloat162float(tmp[i]);
        CK(cudaMemcpy(out, f.data(), (size_t)count * sizeof(float), cudaMemcpyDefault));
        return GALA_OK;
    }
    return fail(c, GALA_EINVAL, "gala_debug_read: unknown selector %d", what);
}

long long gala_launch_count(const gala_ctx* c) { return c ? c->launches : 0; }

int gala_kernel_classes(void) { return T_COUNT; }

const char* gala_kernel_class_name(int k) { return (k >= 0 && k < T_COUNT) ? kTagNames[k] : ""; }

int gala_profile_enable(gala_ctx* c, unsigned long long mask) {
    if (!c) return GALA_EINVAL;
    c->profile_mask = mask;
    return GALA_OK;
}

int gala_profile_read(gala_ctx* c, double* ms, long long* timed, long long* launches, int reset) {
    if (!c) return GALA_EINVAL;
    int r = gala_sync_all(c, -1);
    if (r != GALA_OK) return r;
    for (int k = 0; k < T_COUNT; k++) {
        if (ms) ms[k] = 0.0;
        if (timed) timed[k] = 0;
        if (launches) launches[k] = c->tag_launches[k];
    }
    for (auto& t : c->timed) {
        float f = 0.0f;
        CK(cudaEventElapsedTime(&f, t.beg, t.end));
        if (ms) ms[t.tag] += f;
        if (timed) timed[t.tag]++;
    }
    if (reset) {
        for (auto& t : c->timed) c->event_pool.push_back({t.beg, t.end});
        c->timed.clear();
        for (int k = 0; k < T_COUNT; k++) c->tag_launches[k] = 0;
    }
    return GALA_OK;
}

void* gala_get_stream(gala_ctx* c, int agent) {
    if (!c) return nullptr;
    if (agent < 0) return c->main_stream;
    return agent < c->n ? c->agents[agent].stream : nullptr;
}

const char* gala_last_error(const gala_ctx* c) { return c ? c->err.c_str() : "null context"; }

int gala_gemm_bf16(const void* A, const void* B, float* D, int groups, int M, int N, int K, int a_mn, int b_mn,
                   int split_k, void* stream) {
    if (!A || !B || !D || groups < 1 || M < 1 || N < 1 || K < 1 || split_k < 1) return GALA_EINVAL;
    if ((K % 8) || (a_mn && (M % 8)) || (b_mn && (N % 8))) return GALA_EINVAL;
    if (gemm_init() != cudaSuccess) return GALA_ECUDA;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int bn = N >= 512 ? 256 : b_mn ? (N > 64 ? 128 : 64) : (N > 64 ? 128 : (N > 32 ? 64 : 32));
    GemmOperand oa, ob;
    if (!make_operand(&oa, A, a_mn, M, K, groups, a_mn ? M : K, (uint64_t)M * K, 128)) return GALA_ECUDA;
    if (!make_operand(&ob, B, b_mn, N, K, groups, b_mn ? N : K, (uint64_t)N * K, bn)) return GALA_ECUDA;
    int* err = nullptr;
    if (cudaMalloc(&err, sizeof(int)) != cudaSuccess) return GALA_ENOMEM;
    cudaMemsetAsync(err, 0, sizeof(int), st);
    GemmArgs a;
    memset(&a, 0, sizeof a);
    a.M = M; a.N = N; a.K = K; a.block_n = bn; a.groups = groups; a.split_k = split_k; a.scale = 1.0f;
    a.ldc = N; a.error_word = err;
    int rc = GALA_OK;
    float* ws = nullptr;
    const long count = (long)M * N;
    if (split_k == 1) {
        a.out = D; a.out_group_stride = count;
        if (launch_gemm(oa, ob, a, st) != cudaSuccess) rc = GALA_ECUDA;
    } else {
        if (cudaMalloc(&ws, (size_t)groups * split_k * count * sizeof(float)) != cudaSuccess) { cudaFree(err); return GALA_ENOMEM; }
        a.out = ws; a.out_group_stride = (long)split_k * count; a.out_split_stride = count;
        if (launch_gemm(oa, ob, a, st) != cudaSuccess) rc = GALA_ECUDA;
        if (rc == GALA_OK &&
            launch_splitk_reduce(ws, D, count, split_k, count, groups, (long)split_k * count, count, st) != cudaSuccess)
            rc = GALA_ECUDA;
    }
    // scratch (error word, split-K partials) is released here, so this entry point waits for its work
    if (cudaStreamSynchronize(st) != cudaSuccess) rc = GALA_ECUDA;
    int w = 0;
    if (cudaMemcpy(&w, err, sizeof w, cudaMemcpyDeviceToHost) != cudaSuccess || w) rc = GALA_ECUDA;
    cudaFree(err);
    if (ws) cudaFree(ws);
    return rc;
}

int gala_sweep_sync(float* x, const float* g, float* v, const float* clip, int n_agents, long long d_padded,
                    const gala_topology* topo, long long round, const gala_hparams* hp, void* stream) {
    if (!x || !g || !v || !topo || !hp || n_agents < 1 || d_padded < 4 || (d_padded % 4) || round < 0) return GALA_EINVAL;
    if (topo->kind != GALA_TOPO_RING && topo->kind != GALA_TOPO_EXP) return GALA_EINVAL;
    if (topo->peers < 1 || topo->peers > 2) return GALA_EINVAL;
    int off[2] = {0, 0};
    const int np = topo_offsets(*topo, n_agents, round, off);
    SweepHp s{hp->lr, hp->rms_alpha, hp->rms_eps};
    cudaError_t e = launch_sweep_sync(x, g, v, clip, nullptr, n_agents, d_padded, np, off, s, nullptr,
                                      reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GALA_OK : GALA_ECUDA;
}

int gala_sweep_agents(float* x, const float* g, float* v, float* snap, const float* clip, int n_agents, int n_slots,
                      long long d_padded, const gala_sweep_item* items, int n_items, const gala_hparams* hp, void* stream) {
    if (!x || !v || !snap || !items || !hp || n_agents < 1 || n_slots < 1 || n_items < 0 || d_padded < 4 || (d_padded % 4))
        return GALA_EINVAL;
    if ((long long)n_agents * n_slots > 0x7fffffffLL) return GALA_EINVAL;
    std::vector<char> written((size_t)n_agents * n_slots, 0), listed((size_t)n_agents, 0);
    for (int k = 0; k < n_items; k++) {
        const gala_sweep_item& it = items[k];
        if (it.agent < 0 || it.agent >= n_agents || listed[it.agent] || it.out_slot < 0 || it.out_slot >= n_slots ||
            it.n_peers < 0 || it.n_peers > 2 || (it.has_grad && !g))
            return GALA_EINVAL;
        listed[it.agent] = 1;
        written[(size_t)it.agent * n_slots + it.out_slot] = 1;
    }
    for (int k = 0; k < n_items; k++)
        for (int j = 0; j < items[k].n_peers; j++) {
            const gala_sweep_item& it = items[k];
            if (it.peer[j] < 0 || it.peer[j] >= n_agents || it.peer_slot[j] < 0 || it.peer_slot[j] >= n_slots) return GALA_EINVAL;
            if (written[(size_t)it.peer[j] * n_slots + it.peer_slot[j]]) return GALA_EINVAL;   // read and written in one call
        }
    for (int k0 = 0; k0 < n_items; k0 += kBatch) {
        const int cnt = n_items - k0 < kBatch ? n_items - k0 : kBatch;
        SweepManyArgs a{};
        a.x = x; a.g = g; a.v = v; a.snap = snap; a.clip = clip; a.d_pad = d_padded;
        a.hp = SweepHp{hp->lr, hp->rms_alpha, hp->rms_eps};
        a.n_items = cnt;
        for (int e = 0; e < cnt; e++) {
            const gala_sweep_item& it = items[k0 + e];
            a.it[e].x_row = it.agent;
            a.it[e].out_row = it.agent * n_slots + it.out_slot;
            a.it[e].p_row[0] = it.n_peers > 0 ? it.peer[0] * n_slots + it.peer_slot[0] : -1;
            a.it[e].p_row[1] = it.n_peers > 1 ? it.peer[1] * n_slots + it.peer_slot[1] : -1;
            if (it.has_grad) a.has_grad[e >> 5] |= 1u << (e & 31);
        }
        if (launch_sweep_many(a, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return GALA_ECUDA;
    }
    return GALA_OK;
}

}  // extern "C"
