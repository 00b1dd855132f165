/*
 * marl_actor.h - C ABI of the batched decentralised actor step for multi-agent RL on one GPU.
 *
 * What the library does.  A "worker" in the actor-worker-learner framework (Sec. III-B, Algorithm 2)
 * repeats: get the observations of all of its environments, decide with the shared policy network, send
 * the actions back.  Each environment step is recorded and whole episodes are handed to the learner's
 * replay pool (Algorithm 1 for the hand-over, Algorithm 3 for the learner's side of it).  The hidden state of
 * the recurrent agent is kept per (environment, agent) and never mixed across environments (Sec. III-A,
 * Fig. 3).  This library is that loop for E environments x n agents on the GPU:
 *
 *     x  = [obs | one-hot(agent) | one-hot(last action)]        (last action: none at episode start)
 *     y  = relu(W1 x + b1)
 *     h' = GRUCell(y, h)        r|z|n row blocks, h' = (1-z)*c + z*h, c = tanh(W_in y + b_in + r*(W_hn h + b_hn))
 *     Q  = W2 h' + b2
 *     greedy = lowest available a with Q[a] >= max_avail(Q) - 1e-4f
 *     action = explore ? uniform pick among the available actions : greedy
 *              (Philox4x32-10, counter (step, env, agent, 0), key = seed; explore iff u < eps)
 *     ring[slot_e][pos_e] <- (obs, avail, action, Q, reward, done);  episode end or full slot -> next slot,
 *              h <- 0, last action <- none.
 *
 * The paper names a value-based (Qmix) agent but prints neither its layers nor the exploration rule; the
 * network, the tie rule and the random-number keying above are this library's definition.
 *
 * Conventions
 *   - Every function returns MARL_OK (0) or a negative error code; marl_last_error() gives the text.
 *     Nothing throws or aborts across this boundary.
 *   - "device" pointers are CUDA device addresses on the device that was current at marl_actor_create;
 *     "host" pointers are ordinary process memory.  Borrowed arrays must stay valid until the work
 *     enqueued by the call has finished on the actor's stream; inputs are never written.
 *   - All device work is enqueued on the stream given at creation and is asynchronous unless a function
 *     says that it synchronises.
 *   - Conditions detected on the device (a row with no available action, a bounded wait that expired, an
 *     index out of range) set bits in a status word; a kernel never traps.
 */
#ifndef MARL_ACTOR_H
#define MARL_ACTOR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MARL_OK 0
#define MARL_EINVAL (-1) /* bad argument or configuration */
#define MARL_EALIGN (-2) /* a buffer is not aligned as required (16 bytes) */
#define MARL_ECUDA (-3)  /* a CUDA call failed; marl_last_error() names it */
#define MARL_ENOMEM (-4) /* a caller-provided buffer is too small, or an allocation failed */

#define MARL_PRECISION_FP32 0 /* fp32 weights, fp32 FFMA arithmetic */
#define MARL_PRECISION_BF16 1 /* weight matrices and matmul operands rounded to bf16 (RNE), fp32 accumulate */

#define MARL_KERNEL_AUTO 0   /* bf16: a tensor-core kernel (the pipelined one, else the one-tile one, as the shape allows)
                              * wherever the shape is supported, at every batch size; otherwise, and for fp32, FFMA */
#define MARL_KERNEL_FFMA 1   /* CUDA-core kernel: any shape, both precisions */
#define MARL_KERNEL_TENSOR 2 /* one-tile tcgen05 kernel: bf16 only; create fails if the shape is unsupported */
#define MARL_KERNEL_TENSOR_PIPELINED 3 /* pipelined tcgen05 kernel: bf16, at least 4 agents; hidden 64, or hidden 128
                                        * with at most 16 actions, obs_dim a multiple of 8 and n_agents * n_actions a
                                        * multiple of 16 (weights streamed from L2, dense launches only); create
                                        * fails otherwise.  Inputs that are not 16-byte aligned fall back, per call,
                                        * to the one-tile kernel where the shape allows it, else to the FFMA kernel;
                                        * so do calls whose availability block (batch * n_agents * n_actions bytes)
                                        * is not a 16-byte multiple when an environment's is not, and calls with an
                                        * environment count that is not a multiple of 4 when obs_dim is not a
                                        * multiple of 8 */

#define MARL_MAX_AGENT_TYPES 4

#define MARL_KERNEL_TENSOR_DUAL 4 /* the pipelined design with two tiles of environments resident per SM (never chosen
                                  * automatically: it measures slower than the pipelined kernel): bf16, hidden 64,
                                  * 5 to 32 agents, at most 16 actions, obs_dim a multiple of 8, n_agents * n_actions
                                  * a multiple of 16; create fails otherwise.  Launches it does not take (fewer than 8
                                  * steps, no more tiles than SMs, list steps, unaligned inputs) run on the pipelined
                                  * kernel; results are identical bit for bit */

#define MARL_STATUS_NO_AVAIL 1u  /* some row had no available action (action 0 was taken) */
#define MARL_STATUS_TIMEOUT 2u   /* a bounded device-side wait gave up; results of that launch are invalid */
#define MARL_STATUS_BAD_INDEX 4u /* a ring or state index was out of range and the access was skipped */
/* Bits 8 and above of the status word carry a diagnostic code when MARL_STATUS_TIMEOUT is set (which wait of
 * which warp expired first); they have no meaning otherwise. */

typedef struct marl_actor marl_actor_t; /* opaque; owned by the library; freed by marl_actor_destroy */

/* Dimensions follow Table II of the paper: n agents, A actions, observation width D. */
typedef struct {
  int32_t n_envs;        /* E >= 1 */
  int32_t n_agents;      /* n in [1, 32] */
  int32_t obs_dim;       /* D in [1, 512] */
  int32_t n_actions;     /* A in [1, 32] */
  int32_t hidden;        /* H in {64, 128} */
  int32_t ring_episodes; /* C: episode slots of the replay ring, a positive multiple of E */
  int32_t ring_steps;    /* L: steps per slot; an episode reaching L steps is truncated */
  int32_t precision;     /* MARL_PRECISION_* */
  int32_t kernel;        /* MARL_KERNEL_* */
  int32_t n_agent_types; /* 0 or 1: one network shared by all agents; 2..MARL_MAX_AGENT_TYPES: room for that many
                          * per-type networks (marl_actor_set_weights_typed) */
  uint64_t seed;         /* Philox key of the exploration stream */
  void* stream;          /* cudaStream_t, borrowed; NULL = the legacy default stream */
  /* Device memory.  NULL = the library allocates with cudaMalloc and owns it.  Otherwise the caller's
   * buffer is borrowed until marl_actor_destroy; it must be 256-byte aligned and at least as large as
   * marl_actor_query_sizes reports. */
  void* ring_mem;
  size_t ring_bytes;
  void* state_mem;
  size_t state_bytes;
  void* work_mem;    /* staging for marl_rollout / marl_actor_step_host; may be larger than the minimum: */
  size_t work_bytes; /* marl_rollout stages as many steps per window as fit */
} marl_actor_config_t;

typedef struct {
  size_t ring_bytes;          /* replay ring incl. slot headers */
  size_t state_bytes;         /* recurrent state, counters, status word, packed weights */
  size_t work_bytes_min;      /* staging for one environment step */
  size_t work_bytes_per_step; /* staging per additional step of a rollout window */
} marl_actor_sizes_t;

/* Seeded synthetic environment that stands in for the simulator of Algorithm 1 (Env.step, Env.done).
 * Every stream is a Philox4x32-10 block with counter (step, env, agent | block << 16, tag) and key = seed;
 * tags: 1 done+reward, 2 availability, 3 observation.  A "24-bit threshold" T means: event iff
 * (word >> 8) < T.
 *   done    : word 0 of block 0 of (step, env, agent 0, tag 1) against done_thresh24.
 *   reward  : blocks 1 and 2 of the same stream; the first twelve 16-bit half-words (low half first),
 *             summed, minus 393210, times 2^-16 (an Irwin-Hall stand-in for N(0,1), exact in fp32).
 *   avail   : action 0 always 1; action a > 0: word a%4 of block a/4 of (step, env, agent, tag 2) against
 *             avail_thresh_first (a < avail_split) or avail_thresh_rest.
 *   obs     : law 0: word d%4 of block d/4 of (step, env, agent, tag 3): ((w >> 8) - 2^23) * 2^-23;
 *             law 1: blocks 2d and 2d+1, Irwin-Hall as for the reward, clamped to [-3, 3].
 *             Typed feature blocks: with type_block_len > 0, agents [0, n_type0) are type 0 and the others
 *             type 1; dims [start, start+len) belong to type 0, [start+len, start+2len) to type 1, and an
 *             agent's obs is 0 in the other type's block. */
typedef struct {
  uint64_t seed;
  int32_t obs_law;
  uint32_t done_thresh24;
  uint32_t avail_thresh_first;
  uint32_t avail_thresh_rest;
  int32_t avail_split;
  int32_t n_type0;
  int32_t type_block_start;
  int32_t type_block_len;
} marl_synth_env_t;

/* Replay ring as the learner sees it.  One record per (slot, step) at
 *   base + slot * slot_stride + step * step_stride,
 * fields at the given byte offsets inside the record (each 16-byte aligned):
 *   obs f32[n][D], avail u8[n][A], action i32[n], q f32[n][A] (raw network output, unmasked),
 *   reward f32, done u8.
 * Environment e owns slots e*S .. e*S+S-1 (S = slots_per_env); its k-th episode (k = 0, 1, ...) is written
 * to slot e*S + k%S with id k*E + e.  Headers: slot_epid (-1 = never used), slot_len (steps written),
 * slot_complete (1 once the episode has ended or was truncated at L steps; a truncated episode's last
 * done flag is 0).  All pointers are device addresses, valid until marl_actor_destroy. */
typedef struct {
  void* base;
  size_t slot_stride, step_stride;
  size_t off_obs, off_avail, off_action, off_q, off_reward, off_done;
  int32_t episodes, steps, slots_per_env, n_envs, n_agents, obs_dim, n_actions, reserved;
  int64_t* slot_epid;
  int32_t* slot_len;
  uint8_t* slot_complete;
} marl_ring_view_t;

/* Recurrent state (device arrays) plus the global step counter (host value). */
typedef struct {
  float* h;             /* [E][n][H] */
  int32_t* last_action; /* [E][n], -1 = none */
  int32_t* slot;        /* [E] slot of the open episode */
  int32_t* pos;         /* [E] next position in that slot */
  int64_t* ep_count;    /* [E] episodes closed so far */
  uint64_t step;        /* steps taken since creation / reset: Philox counter word 0 of the next step */
} marl_state_view_t;

typedef struct {
  uint64_t agent_steps; /* rows processed */
  uint64_t episodes;    /* episodes closed (done or truncated) */
  uint64_t explored;    /* rows that took the random branch */
  uint64_t no_avail;    /* rows without any available action */
  uint64_t truncated;   /* episodes closed by the step limit */
} marl_counters_t;

/* Sizes of the three device buffers for a configuration (memory fields of cfg are ignored). */
int marl_actor_query_sizes(const marl_actor_config_t* cfg, marl_actor_sizes_t* out);

/* Creates an actor: validates cfg, carves the buffers, zeroes the state (h = 0, no last action, env e at
 * slot e*S position 0, headers empty, step 0).  Weights are undefined until marl_actor_set_weights.
 * Fails with MARL_ECUDA if no CUDA device is usable: there is no CPU path. */
int marl_actor_create(const marl_actor_config_t* cfg, marl_actor_t** out);

/* Loads the network (Algorithm 2: an iteration starts by fetching the current parameters).  HOST fp32 arrays in
 * [out][in] layout, copied and repacked before the call returns to the caller's stream order:
 *   W1 [H][D+n+A], b1 [H], W_ih [3H][H], b_ih [3H], W_hh [3H][H], b_hh [3H] (row blocks r|z|n),
 *   W2 [A][H], b2 [A].  In bf16 precision the four matrices are rounded to bf16 (RNE); biases stay fp32.
 * version is stored and returned by marl_actor_weights_version. */
int marl_actor_set_weights(marl_actor_t* a, const float* W1, const float* b1, const float* W_ih,
                           const float* b_ih, const float* W_hh, const float* b_hh, const float* W2,
                           const float* b2, uint64_t version);

/* One network per unit type, for heterogeneous teams (Table I of the paper lists a scenario whose team mixes two
 * unit types, and Sec. IV discusses it; the paper's agents share one network, so this is an extension of the
 * worker's decision step of Algorithm 2, not something the paper prints).  Agent i of every environment is decided
 * for by network agent_type[i]; the network input keeps its agent-id one-hot.  HOST arrays: agent_type i32[n], each
 * in [0, n_types); the eight weight arrays as for marl_actor_set_weights with a leading [n_types] axis
 * (W1 [K][H][D+n+A], b1 [K][H], ...).  n_types must not exceed the n_agent_types the actor was created with.
 * Blocking, like marl_actor_set_weights, and a pending publication is dropped.  With n_types > 1 the steps run on
 * the CUDA-core kernel (both precisions; the products are evaluated once per type), marl_actor_publish_weights is
 * refused, and marl_actor_kernel_name reports "ffma"; a later marl_actor_set_weights returns to the shared network
 * and the kernel chosen at creation. */
int marl_actor_set_weights_typed(marl_actor_t* a, int32_t n_types, const int32_t* agent_type, const float* W1,
                                 const float* b1, const float* W_ih, const float* b_ih, const float* W_hh,
                                 const float* b_hh, const float* W2, const float* b2, uint64_t version);

/* The learner's refresh of the shared model while the workers run (Sec. III-B: the learner updates the model in
 * the shared memory pool; Algorithm 2: a worker gets the parameters at the start of an iteration).  The network
 * (HOST arrays as for marl_actor_set_weights, copied before the call returns) becomes the one in use from global
 * step effective_step on (>= the number of steps enqueued so far): the upload runs on a stream of its own beside
 * the steps already enqueued, into the second of two weight images; a later call that spans effective_step runs
 * the steps before it on the old image, makes the stream wait for the upload, swaps the images and runs the rest
 * on the new one - deterministic, whatever the timing.  One publication can be pending: a newer one replaces it,
 * marl_actor_set_weights drops it.  marl_actor_weights_version reports the version of the image in use by the next
 * step to be enqueued. */
int marl_actor_publish_weights(marl_actor_t* a, const float* W1, const float* b1, const float* W_ih,
                               const float* b_ih, const float* W_hh, const float* b_hh, const float* W2,
                               const float* b2, uint64_t version, uint64_t effective_step);
uint64_t marl_actor_weights_version(const marl_actor_t* a);

/* One decision step for all E environments (Algorithm 2, loop body) with recording (Algorithm 1).
 * DEVICE inputs, dense: obs f32[E][n][D], avail u8[E][n][A] (non-zero = available), reward f32[E],
 * done u8[E] - the outcome of this step's joint action, recorded with it.  actions_out i32[E][n] (device)
 * may be NULL.  eps is this step's exploration rate. */
int marl_actor_step(marl_actor_t* a, const float* obs, const uint8_t* avail, const float* reward,
                    const uint8_t* done, float eps, int32_t* actions_out);

/* The step for the environments that have an observation ready (the actors interact with their environments
 * asynchronously, Sec. III-A; the worker serves the observations that have arrived, Algorithm 2): only the M
 * listed environments decide, record and advance; the state and the ring slots of the others are untouched.
 * env_ids i32[M] is a HOST array (the host knows which pipes hold data), copied before the call returns; every
 * entry in [0, E), none twice (MARL_EINVAL otherwise, nothing enqueued).  The other arrays are DEVICE arrays, dense
 * over the list: row x belongs to environment env_ids[x]: obs f32[M][n][D], avail u8[M][n][A], reward f32[M],
 * done u8[M], actions_out i32[M][n] (may be NULL).  The call consumes one index of the global step counter, which
 * keys the exploration stream as (seed, step, environment, agent) with the environment's own index; a trace row
 * of this step is written at the environment's own index as well.  Runs on the pipelined tensor-core kernel where
 * the actor uses it and the arrays can be bulk-copied (16-byte aligned obs and avail), else on the CUDA-core kernel. */
int marl_actor_step_subset(marl_actor_t* a, const int32_t* env_ids, int32_t M, const float* obs,
                           const uint8_t* avail, const float* reward, const uint8_t* done, float eps,
                           int32_t* actions_out);

/* marl_actor_step_subset for environments that answer after the action (Algorithm 1: the actor sends its
 * observation, receives the action and only then steps the environment): prev_reward f32[M] and prev_done u8[M] (device) are the outcome of each listed
 * environment's PREVIOUS action and arrive with this observation.  Per environment, in this order: if a record of
 * the open episode waits for its outcome (cursor > 0), the outcome is written into it and, if the game ended or
 * the slot is full, the episode is closed (header, counters, next slot, zero hidden state, no last action); then
 * the decision on this observation is recorded with reward 0 and done 0 for now.  An environment's first call has
 * nothing waiting: its prev_reward / prev_done are ignored.  Do not mix with the synchronous stepping calls on one
 * actor (they close an episode in the step that ends it).  Kernel choice as for marl_actor_step_subset. */
int marl_actor_step_lagged(marl_actor_t* a, const int32_t* env_ids, int32_t M, const float* obs,
                           const uint8_t* avail, const float* prev_reward, const uint8_t* prev_done, float eps,
                           int32_t* actions_out);

/* The same step with HOST buffers (the observation-action pipe of Algorithms 1 and 2 when the simulators
 * run on the host): copies the four inputs to the device, runs the step, copies the actions back and
 * SYNCHRONISES the stream before returning.  Pinned host memory makes the copies asynchronous. */
int marl_actor_step_host(marl_actor_t* a, const float* obs, const uint8_t* avail, const float* reward,
                         const uint8_t* done, float eps, int32_t* actions_out);

/* Writes n_steps steps of the synthetic environment, starting at step t0, into DEVICE arrays laid out
 * [step][E]...: obs f32[n_steps][E][n][D], avail u8[n_steps][E][n][A], reward f32[n_steps][E],
 * done u8[n_steps][E].  Each array must be 16-byte aligned. */
int marl_env_generate(const marl_actor_t* a, const marl_synth_env_t* env, uint32_t t0, int32_t n_steps,
                      float* obs, uint8_t* avail, float* reward, uint8_t* done);

/* T steps on environment outputs already staged on the device in the layout of marl_env_generate.
 * Step k uses eps = eps_start + (eps_end - eps_start) * min(t, N) / N with t = the global step index and
 * N = anneal_steps (N <= 0: eps_start throughout), evaluated in double and rounded to fp32.
 * Environments are independent, so the kernel may run all T steps of one tile of environments before the
 * next tile; results are those of T calls of marl_actor_step. */
int marl_rollout_staged(marl_actor_t* a, const float* obs, const uint8_t* avail, const float* reward,
                        const uint8_t* done, int32_t T, double eps_start, double eps_end,
                        int32_t anneal_steps);

/* T steps against the synthetic environment: generates windows of steps into the work buffer and runs
 * marl_rollout_staged on each. */
int marl_rollout(marl_actor_t* a, const marl_synth_env_t* env, int32_t T, double eps_start, double eps_end,
                 int32_t anneal_steps);

/* No counterpart in the paper: an integration variant of marl_rollout for callers that cannot allocate
 * device memory - programs that gave all of it to their own pool at start-up, or that must avoid cudaMalloc
 * because it synchronises the device and may fail in the middle of a run.  Same arguments and same results as
 * marl_rollout, but the staging window for the generated environment steps is a fixed array of
 * MARL_NOALLOC_SCRATCH_BYTES inside the library image instead of the actor's work buffer; the function calls no
 * cudaMalloc, cudaFree or other allocating routine.  (Create the actor on caller-provided ring, state and work
 * buffers, otherwise marl_actor_create has already allocated.)
 *   - SET-UP: CUDA loads a library image piece by piece on first use, so the driver places the array on a GPU -
 *     taking that much of its memory until the process exits - during the FIRST call of this function with that
 *     GPU current.  Make that call at start-up, before the remaining device memory goes to your pool and outside
 *     stream capture (the address look-up synchronises); T = 0 does the set-up alone (a and env may be NULL).
 *     Later calls on the device leave the amount of free device memory unchanged;
 *   - MARL_ENOMEM if one environment step of staging (E*n*(4D+A) + 5E bytes plus alignment) exceeds the
 *     array; longer rollouts run in several windows;
 *   - the array is shared by all actors and calls on a device and keeps the previous call's bytes; nothing
 *     in it needs clearing, since each window is fully rewritten before it is read, but calls whose GPU work
 *     overlaps race on it - serialise them.
 * The actor's device must be current, as for every other call.  Error text is not set for the size and
 * look-up failures of this function itself; the return code tells them apart. */
#define MARL_NOALLOC_SCRATCH_BYTES (32u << 20)
int marl_rollout_noalloc(marl_actor_t* a, const marl_synth_env_t* env, int32_t T, double eps_start,
                         double eps_end, int32_t anneal_steps);

/* Optional per-step trace for verification: from the next step on, step k after this call writes its
 * actions to actions[k][E][n] and its Q rows to q[k][E][n][A] (device; either may be NULL) while
 * k < capacity_steps.  Pass NULL, NULL, 0 to switch it off. */
int marl_actor_set_trace(marl_actor_t* a, int32_t* actions, float* q, int32_t capacity_steps);

int marl_ring_view(const marl_actor_t* a, marl_ring_view_t* out);

/* The learner's read of the pool (Algorithm 3: the learner draws a batch of B samples at random from the replay pool; the
 * paper fixes neither the unit nor the law of a sample).  A sample is one complete episode, drawn uniformly and
 * with replacement among the slots whose episode is closed: batch element b of draw number draw_index makes up to
 * MARL_SAMPLE_ATTEMPTS attempts; attempt a takes word 0 of the Philox4x32-10 block with counter
 * (draw_index, b, a, tag 5) and the actor's seed as key, proposes slot floor(w0 * ring_episodes / 2^32) and
 * accepts it if that slot is complete with at least one step.  An element whose attempts all fail is empty
 * (slot -1, length 0, id -1).  The episodes are gathered into a dense batch; steps at and beyond an episode's
 * length are written as zeros.
 * All pointers are DEVICE arrays owned by the caller, 16-byte aligned, written asynchronously on the actor's
 * stream and read by nobody else meanwhile; the ring is only read (a rollout enqueued earlier on the same stream
 * is ordered before the draw).  L = ring_steps. */
#define MARL_SAMPLE_ATTEMPTS 16
typedef struct {
  float* obs;      /* [B][L][n][D] */
  uint8_t* avail;  /* [B][L][n][A] */
  int32_t* action; /* [B][L][n] */
  float* q;        /* [B][L][n][A] */
  float* reward;   /* [B][L] */
  uint8_t* done;   /* [B][L] */
  int32_t* slot;   /* [B] chosen slot or -1 */
  int32_t* len;    /* [B] steps of the episode (0 if empty) */
  int64_t* epid;   /* [B] episode id (k * n_envs + e) or -1 */
} marl_sample_batch_t;
/* Returns MARL_EINVAL for B < 1 or a NULL field, MARL_EALIGN for a misaligned one, MARL_ECUDA if a launch fails. */
int marl_ring_sample(marl_actor_t* a, uint32_t draw_index, int32_t B, const marl_sample_batch_t* out);
int marl_actor_get_state(const marl_actor_t* a, marl_state_view_t* out);
/* Copies the five device arrays of *in into the actor (device-to-device, on the stream) and sets the step
 * counter.  Together with the ring memory this is a checkpoint. */
int marl_actor_set_state(marl_actor_t* a, const marl_state_view_t* in);

/* SYNCHRONISES the stream, then reports and keeps the status bits and counters accumulated so far. */
int marl_actor_status(marl_actor_t* a, uint32_t* device_status, marl_counters_t* counters);

/* Back to the state after creation (weights are kept).  Asynchronous. */
int marl_actor_reset(marl_actor_t* a);

/* SYNCHRONISES the stream and frees what the library allocated. */
void marl_actor_destroy(marl_actor_t* a);

/* Failure-detection self-test (no counterpart in the paper): launches a one-block kernel that waits, with the
 * bounded wait the tensor-core kernel uses for all of its hand-offs, on a barrier that nothing completes.  The
 * wait gives up after poll_limit polls (1 .. 1000000; 20000 is a few tens of milliseconds) and the kernel
 * reports it.  SYNCHRONISES the stream.  *status_out (host) receives MARL_STATUS_TIMEOUT | 0x100 when the
 * mechanism works.  The CUDA context stays usable afterwards. */
int marl_selftest_bounded_wait(void* stream, uint32_t poll_limit, uint32_t* status_out);

/* Measurement helper (no counterpart in the paper): runs a dependency-free fp32 FMA loop on every SM and reports
 * the best of three timed repetitions in TFLOP/s - the arithmetic bound of the fp32 actor path on this device
 * at the clocks it actually sustains.  SYNCHRONISES the stream; takes a few tens of milliseconds. */
int marl_measure_ffma_tflops(void* stream, double* tflops_out);

/* Name of the step kernel in use: "ffma", "tcgen05" (one-tile tensor-core kernel), "tcgen05-pipelined",
 * "tcgen05-dual" (two resident tiles; its other launches run on the pipelined kernel), or
 * "tcgen05-streamed" (hidden size 128: the pipelined design with the weights streamed through shared memory). */
const char* marl_actor_kernel_name(const marl_actor_t* a);

/* Launches of library kernels enqueued by this actor since creation (all kernels, all entry points). */
uint64_t marl_actor_launch_count(const marl_actor_t* a);

/* Text of the last error on the calling thread ("" if none). */
const char* marl_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MARL_ACTOR_H */
