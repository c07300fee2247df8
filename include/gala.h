/*
 * gala.h -- C ABI of the B200 learner library for GALA-A2C
 * (Gossip-based Actor-Learner Architectures, arXiv 1906.04585).
 *
 * The library holds N co-resident actor-learners ("agents") on one GPU and
 * runs, per agent, the steps of Algorithm 1 after the environment
 * interaction: network forward/backward over a rollout, n-step returns,
 * advantages and the A2C objective, RMSProp, and the gossip average with the
 * agent's in-peers.  Every step runs in CUDA kernels built for sm_100a; there
 * is no CPU fallback.
 *
 * Conventions
 *  - Every call returns 0 (GALA_OK) or a negative gala_status.  After a
 *    failure, gala_last_error(ctx) returns a library-owned message that stays
 *    valid until the next call on that context.
 *  - The context owns parameters, optimiser state, snapshots, workspaces,
 *    CUDA streams and events.  Rollout / observation / output buffers are
 *    DEVICE pointers owned by the caller; they must stay valid until the
 *    agent's stream has passed the call (gala_sync_agent, or gala_sync_all).
 *    The only HOST pointers are the structs, gala_in_peers / gala_losses /
 *    gala_stats outputs, and gala_get_state / gala_set_state buffers, which
 *    may be host or device memory (the library asks the CUDA runtime which).
 *  - Calls enqueue work and return; only the sync and get/set-state calls
 *    wait.  One host thread per context.
 *  - No kernel traps or spins without a bound.  A device-side wait that runs
 *    out sets an error word that the next sync call reports as GALA_ECUDA.
 *
 * Flat parameter vector of one agent (x_i = (omega_i, theta_i), Sec. 3),
 * float32, d entries, padded to d_padded:
 *   conv net (Appendix C.2: 3 conv layers, one hidden layer, linear heads;
 *   84x84x4 input, NHWC):
 *     conv1.W[32][8][8][4]  conv1.b[32]      stride 4
 *     conv2.W[64][4][4][32] conv2.b[64]      stride 2
 *     conv3.W[64][3][3][64] conv3.b[64]      stride 1
 *     fc.W[512][7][7][64]   fc.b[512]
 *     pi.W[A][512] pi.b[A]  v.W[1][512] v.b[1]
 *   MLP:  l1.W[H][obs_dim] l1.b[H]  l2.W[H][H] l2.b[H]
 *         pi.W[A][H] pi.b[A]  v.W[1][H] v.b[1]
 *   i.e. output-channel major, then (kh, kw, cin): the reduction index is the
 *   fastest one.
 */
#ifndef GALA_H
#define GALA_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gala_ctx gala_ctx; /* opaque */

typedef enum {
    GALA_OK = 0,
    GALA_EINVAL = -1,   /* bad argument; nothing was enqueued */
    GALA_ENOMEM = -2,   /* device or host allocation failed */
    GALA_ECUDA = -3,    /* CUDA runtime error or device-side error word set */
    GALA_ETIMEOUT = -4, /* a host wait with a deadline ran out */
    GALA_ESTATE = -5    /* call not valid in the context's current state */
} gala_status;

typedef enum { GALA_NET_MLP = 0, GALA_NET_CONV = 1 } gala_net_kind;

typedef struct {
    int kind;       /* gala_net_kind */
    int obs_dim;    /* MLP: observation length (float32). CONV: ignored (84x84x4 uint8) */
    int hidden;     /* MLP: width of the two tanh layers. CONV: ignored (512) */
    int n_actions;  /* 2..32 */
    int gemm_dtype; /* 0 = fp32 FMA (MLP), 1 = bf16 operands, fp32 accumulate (CONV) */
} gala_net_spec;

typedef enum { GALA_TOPO_RING = 0, GALA_TOPO_EXP = 1, GALA_TOPO_COMPLETE = 2 } gala_topo_kind;

/* Communication topology = the non-zero pattern of the mixing matrix P^(k)
 * (Sec. 2 "Gossip algorithms", Sec. 3).  Non-zero weights are 1/(1+|N_in_i|)
 * (footnote of Algorithm 1).
 *   RING: directed ring v_0 -> v_1 -> ... -> v_{n-1} -> v_0 (Appendix C.2,
 *         Fig. 5); in-peers of i are i-1 .. i-peers (mod n).
 *   EXP:  time-varying exponential graph, L = ceil(log2 n): the j-th in-peer
 *         of i at round k is i - 2^((peers*k + j) mod L) (mod n).
 *   COMPLETE: the synchronous A2C baseline of Sec. 5 (agents average their GRADIENTS before each
 *         update, equivalent to one agent with all simulators): only gala_step_sync is defined;
 *         `peers` is ignored; gala_gossip and gala_in_peers refuse. */
typedef struct {
    int kind;  /* gala_topo_kind */
    int peers; /* in-peers per round: 1 or 2 */
} gala_topology;

/* Hyper-parameters (Table 2).  lr is used as given (the sqrt(#learners)
 * scaling of Table 2 is the caller's). */
typedef struct {
    float lr;            /* 7e-4 */
    float rms_alpha;     /* RMSProp decay, 0.99 */
    float rms_eps;       /* added outside the square root */
    float gamma;         /* discount, 0.99 */
    float ent_coef;      /* eta of Eq. 3, 0.01 */
    float vf_coef;       /* weight of the TD loss of Eq. 1, 0.5 */
    float max_grad_norm; /* global-norm clip, 0.5; <= 0 switches it off */
    int n_envs;          /* E: simulators per agent */
    int n_steps;         /* T: rollout horizon (N in the paper) */
    int staleness_tau;   /* tau of Sec. 3: < 0 unbounded; >= 0: a gossip step that finds no fresh message
                            after more than tau local iterations without one waits for its in-peers */
    unsigned long long seed; /* initial parameters (library's own generator) */
    int identical_init;  /* 1: all agents start from the same parameters (assumed by Prop. 1) */
} gala_hparams;

/* One agent's rollout {(s_t, a_t, r_t, s_{t+1})} (Algorithm 1, acting step). DEVICE pointers. */
typedef struct {
    const void* obs;            /* [T+1][E][84][84][4] uint8 (16-byte aligned)  or  [T+1][E][obs_dim] float32 */
    const int* actions;         /* [T][E], each in [0, n_actions) */
    const float* rewards;       /* [T][E] */
    const unsigned char* dones; /* [T][E]; 1 = the episode ended at this step */
} gala_rollout;

/* Create n_agents agents (1..256).  Allocates everything; parameters are
 * initialised from hp->seed (uniform +-1/sqrt(fan_in)), square-average state
 * to 0, round counters to 0.  Uses the current CUDA device.
 * Environment variables read here select older or alternative kernels for the same results; they exist so that
 * two independent implementations can be compared with each other and with the CPU oracle:
 *   GALA_HEADS_UNFUSED   separate kernels for heads, objective and head gradients
 *   GALA_MLP_UNFUSED     separate kernels for the small fully connected network
 *   GALA_C1B_SLICES=0/1  conv1's bias gradient from column sums of dY1 / from conv2's data-gradient kernel
 *                        (default: the latter for launches over at least 2048 samples)
 *   GALA_FC_BN=128/256   columns of an output tile of the hidden layer's forward product
 * A build of the same sources with GALA_CROSS_CHECK defined (libgala_check.so, loaded by one test only) also knows
 *   GALA_CONV_LEGACY     convolution products with one tensor copy per kernel offset and bf16 frame copies */
int gala_create(int n_agents, const gala_topology* topo, const gala_net_spec* net,
                const gala_hparams* hp, gala_ctx** out);
int gala_destroy(gala_ctx* ctx);

/* Acting step of Algorithm 1: forward on E observations obs[E][...], softmax,
 * inverse-CDF draw a = min{k : sum_{j<=k} pi_j > u} (clamped to A-1) from the
 * caller's uniforms[E] in [0,1); writes actions[E] (int32), values[E].  All
 * DEVICE pointers; actions or values may be NULL.  Uses the agent's forward
 * workspace: do not interleave between gala_learn and its completion on
 * another stream. */
int gala_act(gala_ctx* ctx, int agent, const void* obs, const float* uniforms, int* actions,
             float* values);

/* Learner step of Algorithm 1 (returns, advantages, A2C gradient; Eqs. 1-4)
 * on the agent's stream.  Leaves a pending gradient and its global norm.  If a
 * gradient is already pending it is first applied without mixing (the
 * no-gossip update of the appendix) and published. */
int gala_learn(gala_ctx* ctx, int agent, const gala_rollout* rollout);

/* Optimiser + gossip steps of Algorithm 1 on the agent's stream, one fused
 * pass over the flat vector: RMSProp with the pending gradient (none
 * pending: parameters unchanged), publish the result as the agent's newest
 * snapshot (the non-blocking broadcast), and, if a snapshot newer than the
 * one last consumed has COMPLETED for every in-peer of the agent's current
 * round, replace the parameters by the equal-weight average (Eq. 6);
 * otherwise keep the local result (Eq. 5).  Never waits for a peer. */
int gala_gossip(gala_ctx* ctx, int agent);

/* The learner step of Algorithm 1 for SEVERAL agents whose rollouts have arrived, as one set of grouped launches
 * (every kernel of the step works on the whole list; the kernels are those of gala_step_sync), without any of
 * the listed agents waiting for an agent that is not listed (Sec. 3: agents proceed at their own pace).
 * agents[m]: distinct agent indices in any order; rollouts[m]: rollouts[k] belongs to agents[k].  Per agent the
 * call is gala_learn: a gradient that is still pending is first applied without mixing and published.  The work
 * goes to one of two internal streams; the call orders it behind everything enqueued for the listed agents
 * before, and later per-agent calls for them behind it.  A host that polls which simulators have delivered and
 * hands the ready agents to this call amortises the launch cost of a step over all of them.  Networks other
 * than the conv net (and rollouts too long for the fused heads kernel) are handled as m calls of gala_learn. */
int gala_learn_many(gala_ctx* ctx, const int* agents, const gala_rollout* rollouts, int m);

/* gala_gossip for several agents in one launch: for every listed agent the RMSProp step with its pending
 * gradient, the broadcast of the result as its newest snapshot and, where a snapshot newer than the one last
 * consumed has COMPLETED for each of its in-peers, the equal-weight average (Eqs. 5-6).  Which snapshots are
 * usable - complete, or published by an earlier grouped call on the same internal stream and therefore complete
 * before this call's launch runs - is decided for the whole list before anything is enqueued, so a listed agent
 * never sees a snapshot published by the same call; listed agents that are each other's in-peers are fine (three snapshot slots per
 * agent: the slot being written is never one that may be read).  Per-agent results, counters and gala_last_mix
 * are as after m calls of gala_gossip.  GALA_ETIMEOUT from the staleness bound: nothing was enqueued. */
int gala_gossip_many(gala_ctx* ctx, const int* agents, int m);

/* Streams the grouped calls alternate between: 1 (default) or 2.  With one, grouped calls run on the device in
 * the order they were made, every kernel's set-up overlapping its predecessor's tail also across calls, and a
 * gossip step sees every snapshot that an earlier grouped call published (it runs after it).  With two, the
 * launch sets of consecutive gala_learn_many calls may overlap on the device; a snapshot published on the other
 * stream counts only once it has completed. */
int gala_set_group_lanes(gala_ctx* ctx, int lanes);

/* Non-blocking: *busy = 0 when the agent's latest optimiser / gossip step, and whatever was enqueued for the agent
 * after it, has completed on the device; 1 otherwise.  For hosts that hand the next rollout of an agent to
 * gala_learn_many only when the parameters it was collected with are in place. */
int gala_poll_agent(gala_ctx* ctx, int agent, int* busy);

/* Straggler injection for experiments (the slow simulators of Sec. 1 / Sec. 5 "computational
 * performance"): keeps the agent's stream busy for about `usec` microseconds (0..100000) with one
 * sleeping thread before whatever is enqueued next on it.  The wait is bounded on the device. */
int gala_delay(gala_ctx* ctx, int agent, int usec);

/* Deterministic synchronous round for all agents (Eq. 7 with zero delay):
 * learn on rollouts[0..n_agents), then x_i <- (y_i + sum_{j in N_in_i(k)} y_j)/(1+p)
 * with y the post-RMSProp parameters of the SAME round.  Runs on the
 * context's main stream; waits for all agent streams first.  rollouts may be
 * NULL: then the gradients currently stored (gala_set_grad) are used. */
int gala_step_sync(gala_ctx* ctx, const gala_rollout* rollouts);

/* Host waits.  timeout_ms < 0: no deadline.  GALA_ETIMEOUT if work is still
 * running at the deadline (nothing is cancelled). */
int gala_sync_agent(gala_ctx* ctx, int agent, int timeout_ms);
int gala_sync_all(gala_ctx* ctx, int timeout_ms);

/* Schedule query (host integers): in-peers of `agent` at round `round`.
 * peers[] needs room for topo.peers entries. */
int gala_in_peers(const gala_ctx* ctx, long long round, int agent, int* peers, int* n);

/* State exchange (synchronises the agent first).  Any pointer may be NULL.
 * Buffers hold d floats (not padded); host or device memory. */
int gala_get_state(gala_ctx* ctx, int agent, float* params, float* sq_avg, float* grad,
                   long long* round);
int gala_set_state(gala_ctx* ctx, int agent, const float* params, const float* sq_avg,
                   long long round);
/* Store a gradient as the agent's pending gradient (for optimiser-only runs).
 * clip_coef is the factor c applied to it (1 = none); < 0: compute it from
 * max_grad_norm on the device. */
int gala_set_grad(gala_ctx* ctx, int agent, const float* grad, float clip_coef);

/* Distance of the agents' parameters from their mean, ||X - mean||_F over all agents and
 * parameters (left-hand side of Propositions 1 and 2).  Waits for all work first. */
int gala_consensus_distance(gala_ctx* ctx, double* out);
/* Update norms for the bound of Proposition 1, ||X - mean||_F <= alpha * sum_s beta^(k+1-s) ||G(s)||.
 * gala_track_updates(ctx, 1): every later gala_step_sync also computes, before its optimiser pass and from the same
 * gradient, clip factor and second-moment estimate, the Frobenius norm over all agents of the step it takes
 * (row i = lr * c g / (sqrt(v') + eps), i.e. alpha G of that round); one more kernel that reads g and v once,
 * off by default.  gala_update_norm waits for the main stream and returns the value of the last such round;
 * GALA_EINVAL when there has been none. */
int gala_track_updates(gala_ctx* ctx, int on);
int gala_update_norm(gala_ctx* ctx, double* out);
/* Longest host wait (ms, default 1000) of a gossip step that is blocked by the staleness bound.
 * When it runs out, or when an in-peer has published nothing newer, gala_gossip returns
 * GALA_ETIMEOUT and has enqueued nothing; the pending gradient stays pending. */
int gala_set_stale_timeout(gala_ctx* ctx, int timeout_ms);
/* SM budget of one agent's tensor-core kernels in the per-agent calls (gala_learn, gala_act): at most `ctas`
 * thread blocks per kernel, so that kernels of several agents' streams run side by side instead of each
 * taking every SM in turn (Sec. 3: the agents progress independently).  0 or at least the device's SM count: no
 * limit (default at creation: 8 x SM count / n_agents, at least 32, no limit for fewer than 5 agents).  gala_step_sync is not
 * affected.  Results do not depend on the budget except through the summation order of sliced weight
 * gradients. */
int gala_set_agent_ctas(gala_ctx* ctx, int ctas);
/* Closed actor loop for one agent, enqueued on its stream without a host wait (Algorithm 1, whole loop body):
 * `iterations` times { T times: act on the current observations of the agent's E environments, step the
 * environments with the sampled actions and store the transition; then gala_learn on the stored rollout and
 * gala_gossip }.  The environments are a synthetic stand-in for the paper's simulators (which run on CPUs and
 * are no part of this library): a counter-based function of (env_seed, agent, environment, step) on the SplitMix64
 * output function sm(z): z += 0x9E3779B97F4A7C15; z = (z ^ z >> 30) * 0xBF58476D1CE4E5B9; z = (z ^ z >> 27) *
 * 0x94D049BB133111EB; return z ^ z >> 31.  With base = sm(sm(sm(env_seed + agent) + environment) + step):
 * the uniform of the action draw is (sm(base + (3 << 56)) >> 40) * 2^-24; a frame's byte j is byte j % 8
 * (little-endian) of sm(base + j / 8), a float observation's element j is ((sm(base + j) >> 40) * 2^-23 - 1) *
 * sqrt(3); the reward is 1 when the action equals sm(base + (1 << 56)) mod n_actions, else 0; the episode ends
 * when sm(base + (2 << 56)) >> 40 < 167772 (probability 0.01).  Steps are numbered per agent from 0 and continue over
 * calls.  The rollout buffers belong to the library (allocated by the first call for an agent).  Unless graph
 * replay is off (gala_set_graphs), an agent's iteration without its gossip step is captured on its second run
 * and replayed as one graph launch from the third on.  Returns as
 * gala_learn / gala_gossip do (GALA_ETIMEOUT from a staleness-bounded gossip step ends the loop early). */
int gala_actor_loop(gala_ctx* ctx, int agent, int iterations, unsigned long long env_seed);
/* The same loop for ALL agents in lockstep (Algorithm 1 with the agents advancing together, as in the synchronous
 * round): `iterations` times { T times: one forward pass over the E current observations of every agent, then one
 * kernel that draws every agent's actions and steps every agent's environments; then gala_step_sync on the stored
 * rollouts }.  Same environment function, same step counters and same rollout buffers as gala_actor_loop (the two
 * may alternate); acting is batched over the agents, so an iteration is some 50 launches however many agents there
 * are.  The acting part is captured on its second run and replayed as one graph launch from the third on (unless
 * graph replay is off); the round inside follows gala_step_sync's own rule.  Returns as gala_step_sync does;
 * GALA_ESTATE with the earlier convolution kernels (cross-check build only). */
int gala_actor_loop_all(gala_ctx* ctx, int iterations, unsigned long long env_seed);
/* Waits for the agent's stream and copies the rollout of its last loop iteration to HOST memory (any pointer
 * may be NULL): obs [T+1][E][...], actions [T][E], rewards [T][E], dones [T][E]; *next_step = number of
 * environment steps taken so far. */
int gala_actor_read(gala_ctx* ctx, int agent, void* obs, int* actions, float* rewards, unsigned char* dones,
                    long long* next_step);
/* CUDA-graph replay of the learner step.  mode 1 (default): in gala_step_sync; 2: also in gala_learn; 0: never.
 * The first call with a given set of rollout buffers launches its kernels one by one; the second captures the
 * same launches into a graph; from then on the step is one graph launch (the kernels and their results are the
 * same).  A caller that reuses its rollout buffers, as an actor that writes each rollout into the same device
 * memory does, gets this for every step; one that passes new buffers every time never pays for a capture.  Up to
 * 512 distinct buffer sets are remembered.  Instantiating a graph costs about a millisecond of host time, which
 * pays off in the synchronous round (host-bound at small batches) and not in the per-agent calls of many agents
 * (bound by the device; 64 agents x 4 buffer sets are 256 graphs), hence the default.  Off while per-class timing
 * (gala_profile_enable) of a kernel inside the step is on.  If the application itself captures the library's
 * streams into a graph, switch this off first. */
int gala_set_graphs(gala_ctx* ctx, int mode);
int gala_param_count(const gala_ctx* ctx, long long* d, long long* d_padded);
/* out = {policy term, mean squared TD error, mean entropy, gradient norm} of the last learn. */
int gala_losses(gala_ctx* ctx, int agent, float out[4]);
/* The same four numbers for every agent, out[agent][4] (host memory, 4 * n_agents floats): one wait and two
 * copies instead of two per agent. */
int gala_losses_all(gala_ctx* ctx, float* out);
/* out = {frames, rounds, mixes, skipped mixes, staleness sum, staleness max, published version,
 *        gossip steps that waited because of the staleness bound} */
int gala_stats(gala_ctx* ctx, int agent, long long out[8]);
/* Which snapshot versions the agent's last gala_gossip consumed: versions[j]
 * for in-peer peers[j]; *mixed = 1 if the average was taken. */
int gala_last_mix(gala_ctx* ctx, int agent, int* peers, long long* versions, int* n, int* mixed);
/* Read snapshot `version` of an agent if it is still held (the two newest are; an agent has three slots, the
 * third being the one its next publication goes to). */
int gala_get_snapshot(gala_ctx* ctx, int agent, long long version, float* out);
/* Adopt a caller's CUDA stream (cudaStream_t) for the agent; NULL restores the library's. */
int gala_set_stream(gala_ctx* ctx, int agent, void* cuda_stream);
/* Copy intermediate tensors of the last learn/act of an agent for checks:
 * what = 0 logits [B][A] f32, 1 values [B] f32, 2 returns [S], 3 advantages [S],
 * 4 dlogits [S][A], 5 dvalues [S]; 10+l: output of trunk layer l as float32
 * (B = (T+1)E rows); 20: the bf16 copy of the agent's parameters that the conv
 * net's products read, as float32 [d].  out: host or device, `count` floats. */
int gala_debug_read(gala_ctx* ctx, int agent, int what, float* out, long long count);
/* Failure reporting, exercised without a failure: enqueues on the agent's stream a one-thread kernel that waits,
 * with the bounded wait of the tensor-core kernels limited to `polls` polls (1..100000, microseconds in all), on a
 * barrier that nothing arrives at, gives up and raises the context's error word exactly as those kernels do when
 * a wait of theirs runs out.  The next gala_sync_agent / gala_sync_all / gala_get_state then returns GALA_ECUDA
 * ("a bounded device-side wait ran out") and clears the word; the context stays usable. */
int gala_debug_wait_runs_out(gala_ctx* ctx, int agent, int polls);
/* Number of kernel launches issued by this context so far. */
long long gala_launch_count(const gala_ctx* ctx);
/* Kernel classes (im2col, each GEMM, sweeps, ...) for per-class accounting. */
int gala_kernel_classes(void);
const char* gala_kernel_class_name(int k);
/* Bracket every launch of the classes in `mask` (bit k = class k) with CUDA timing events on the
 * launching stream; 0 switches timing off.  Launch counts per class are always kept. */
int gala_profile_enable(gala_ctx* ctx, unsigned long long mask);
/* Waits for all work, then fills per class (arrays of gala_kernel_classes() entries, any may be
 * NULL): summed device time in ms of the timed launches, how many launches were timed, and how
 * many were issued since the last reset.  reset != 0 clears the counters and recorded events. */
int gala_profile_read(gala_ctx* ctx, double* ms, long long* timed, long long* launches, int reset);
/* The CUDA stream (cudaStream_t) an agent's work is enqueued on; agent < 0: the stream of the
 * synchronous mode.  Owned by the library unless set by gala_set_stream. */
void* gala_get_stream(gala_ctx* ctx, int agent);
const char* gala_last_error(const gala_ctx* ctx);

/* Stand-alone grouped GEMM on the tensor cores, exposed for validation:
 * D[g] = op(A[g]) * op(B[g])^T, bf16 operands, fp32 accumulate, fp32 output
 * D[g][M][N] row-major.  a_mn = 0: A stored [M][K] (K contiguous); 1: stored
 * [K][M].  b_mn = 0: B stored [N][K]; 1: stored [K][N].  DEVICE pointers to
 * bf16 (A, B) and float (D); K, M, N and the leading dimensions must keep
 * rows 16-byte aligned (multiples of 8 elements).  split_k >= 1 splits the
 * reduction and sums the partials in a fixed order.  Runs on `stream`
 * (cudaStream_t, may be NULL); allocates its scratch with cudaMalloc, waits for
 * its work and frees the scratch before it returns. */
int gala_gemm_bf16(const void* A, const void* B, float* D, int groups, int M, int N, int K,
                   int a_mn, int b_mn, int split_k, void* stream);

/* gala_gemm_bf16 without any allocation (this entry point has no counterpart in the paper; it
 * exists for the way the library gets embedded).  gala_gemm_bf16 obtains its split-K scratch with
 * cudaMalloc / cudaFree.  Some hosts of this library cannot afford that: a process in which a
 * framework's caching allocator already holds almost all device memory (the allocation may simply
 * fail), or a serving / control loop with a fixed memory plan, where the device-wide
 * synchronisation inside cudaMalloc and cudaFree stalls every other stream.  This variant computes
 * the same product -- same arguments, same kernels, same summation order -- but keeps its scratch
 * in an 8 MiB array built into the library image (held by every GPU that loads the library, from
 * load until exit) and calls no allocating routine.
 *   Limit: groups * split_k * M * N <= 2 Mi floats when split_k > 1; beyond that the call is
 *   refused with GALA_EINVAL and a message naming the limit (no limit for split_k == 1).
 *   First call on each device: looks up the array's device address, resolves the tensor-map
 *   encoder and opts the kernel in to large shared memory on that device; make that first call
 *   before any stream capture begins.  Every call waits on `stream` for its own work (and reads
 *   one status word back on that stream) before it returns; it waits for no other stream.
 *   All calls share the one array, which keeps the previous call's contents (the call clears the
 *   only word that must start at zero).  Two calls whose GPU work overlaps -- different streams,
 *   threads or processes' contexts on the same device and library image -- race on it; this entry
 *   point waits for its own work before returning, so successive calls from one thread are safe.
 * errbuf (may be NULL) receives a NUL-terminated message of at most errbuf_len bytes on failure.
 * Returns GALA_OK, GALA_EINVAL or GALA_ECUDA. */
int gala_gemm_bf16_static(const void* A, const void* B, float* D, int groups, int M, int N, int K,
                          int a_mn, int b_mn, int split_k, void* stream, char* errbuf, int errbuf_len);

/* Stand-alone fused RMSProp + gossip pass over caller-owned arrays, exposed
 * for the optimiser micro-benchmark and its parity test (Algorithm 1 optimiser
 * and gossip steps; Eq. 7).  x, g, v: DEVICE float32 [n_agents][d_padded],
 * updated in place (x, v).  Synchronous all-agent form: every agent takes its
 * RMSProp step and all mix simultaneously with the in-peers of `round`.
 * clip: DEVICE float[n_agents] or NULL (= 1).  d_padded % 4 == 0. */
int gala_sweep_sync(float* x, const float* g, float* v, const float* clip, int n_agents,
                    long long d_padded, const gala_topology* topo, long long round,
                    const gala_hparams* hp, void* stream);

/* Stand-alone per-agent form of the fused RMSProp + gossip pass for a list of agents in ONE launch per 64 agents
 * (Algorithm 1: optimiser step, broadcast, conditional average; Eqs. 5-6), over caller-owned DEVICE arrays:
 * x, g, v float32 [n_agents][d_padded]; snap float32 [n_agents][n_slots][d_padded] (the agents' published
 * snapshots); clip float[n_agents] or NULL (= 1).  For item k (distinct agents):
 *   y = RMSProp(x, clip * g, v) if has_grad, else y = x (v untouched);  snap[agent][out_slot] = y;
 *   x = (y + sum_j snap[peer[j]][peer_slot[j]]) / (1 + n_peers)     (n_peers = 0: x = y).
 * No snapshot slot may be both read and written by one call (GALA_EINVAL).  Bytes per parameter and agent:
 * 24 + 4 n_peers (x, g, v and the peers' snapshots read once; x, v and the own snapshot written once).
 * d_padded % 4 == 0; every array 16-byte aligned.  Enqueues on `stream` and returns. */
typedef struct {
    int agent;
    int out_slot;
    int n_peers;      /* 0..2 */
    int peer[2];
    int peer_slot[2];
    int has_grad;
} gala_sweep_item;
int gala_sweep_agents(float* x, const float* g, float* v, float* snap, const float* clip, int n_agents, int n_slots,
                      long long d_padded, const gala_sweep_item* items, int n_items, const gala_hparams* hp,
                      void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GALA_H */
