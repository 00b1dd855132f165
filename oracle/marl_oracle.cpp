// CPU oracle for the batched decentralised actor step.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, scalar statement of what the actor path
// computes.  It shares no code, header, table or constant with the CUDA library and is never on the
// product path: only the test-suite, the smoke check and the benchmark's CPU-baseline leg load it.
//
// What it follows
//   * Control flow: the worker loop of Algorithm 2 (get observations of every actor, decide with the
//     policy network, send the actions back) and the actor loop of Algorithm 1 (reset at episode
//     start, one observation/action exchange per environment step, the whole track handed over when
//     the episode ends).
//   * Hidden state: one vector per (environment, agent), never mixed across environments
//     (Sec. III-A, Fig. 3).
//   * Replay pool: every step is recorded and whole episodes become visible to the learner
//     (Sec. III-B; Algorithm 1 hands the finished track over, Algorithm 3 files it in the pool).
//   * The paper does not print the agent network (it only says "value-based"/Qmix, Sec. III and
//     Sec. IV-B).  The network here is the usual recurrent Qmix agent:
//       x = [obs | one-hot(agent id) | one-hot(last action)]  ->  Linear(H) -> ReLU -> GRUCell(H)
//         -> Linear(A),
//     with the textbook GRU cell
//       r = sigmoid(W_ir y + b_ir + W_hr h + b_hr)
//       z = sigmoid(W_iz y + b_iz + W_hz h + b_hz)
//       c = tanh  (W_in y + b_in + r * (W_hn h + b_hn))
//       h' = (1 - z) * c + z * h
//     and row blocks r | z | n inside W_ih and W_hh.
//   * Random numbers: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11), written here from
//     its published definition.
//
// Arithmetic: every dot product accumulates in double, sequentially, bias first.  exp and tanh are the
// C library's double versions.  Values that the method *stores* (Q, hidden state) are rounded to float
// when stored, because the next step consumes the stored value.  The "bf16" mode rounds the weight
// matrices and the four matrix-multiply operands (observation, fc1 output, hidden state as the W_hh
// operand, new hidden state as the fc2 operand) to bfloat16, round-to-nearest-even; everything else is
// unchanged.
//
// Pins (tests marked "not gpu"): Philox known-answer vectors; closed-form GRU cases (zero weights,
// saturated gates, scalar network); float64 library Linear/GRUCell; brute-force masked arg-max over all
// masks; statistical checks of the epsilon draw and of every synthetic-environment stream; ring
// invariants.  The composition of a whole rollout has no external reference: "parity unpinned" beyond
// the pins of its parts and the invariants.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC (no intrinsics, no fast-math).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <sched.h>
#include <thread>
#include <vector>

namespace {

// ---------------------------------------------------------------------------------------------------
// Philox4x32-10.  One round maps the counter (c0,c1,c2,c3) with round key (k0,k1) to
//   (hi(M1*c2) ^ c1 ^ k0,  lo(M1*c2),  hi(M0*c0) ^ c3 ^ k1,  lo(M0*c0)),
// and the key is advanced by the Weyl constants between rounds (nine advances for ten rounds).
// ---------------------------------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint64_t M0 = 0xD2511F53ull, M1 = 0xCD9E8D57ull;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) { k0 += W0; k1 += W1; }
    const uint64_t p0 = M0 * (uint64_t)c0;
    const uint64_t p1 = M1 * (uint64_t)c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Stream tags (counter word 3).
enum : uint32_t { TAG_EPS = 0, TAG_DONE_REWARD = 1, TAG_AVAIL = 2, TAG_OBS = 3 };

// Counter layout: (step, env, agent | block << 16, tag); key = (seed low word, seed high word).
void philox_block(uint64_t seed, uint32_t step, uint32_t env, uint32_t agent, uint32_t block,
                  uint32_t tag, uint32_t out[4]) {
  const uint32_t ctr[4] = {step, env, agent | (block << 16), tag};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  philox4x32_10(ctr, key, out);
}

// 24-bit uniform in [0,1): exact in float.
float uniform24(uint32_t w) { return (float)(w >> 8) * (1.0f / 16777216.0f); }

// round-to-nearest-even float -> bfloat16 -> float
float bf16_round(float x) {
  uint32_t u;
  std::memcpy(&u, &x, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return x;  // NaN passes through
  const uint32_t keep_lsb = (u >> 16) & 1u;
  u += 0x7FFFu + keep_lsb;
  u &= 0xFFFF0000u;
  float y;
  std::memcpy(&y, &u, 4);
  return y;
}

// Sum of 12 uniform 16-bit integers, centred and scaled: mean 0, variance 1 - 2^-32, support about +-6.
// Every value is a multiple of 2^-16 below 2^3 in magnitude, hence exact in float.
float irwin_hall12(const uint32_t a[4], const uint32_t b[4]) {
  int64_t s = 0;
  for (int k = 0; k < 4; ++k) s += (int64_t)(a[k] & 0xFFFFu) + (int64_t)(a[k] >> 16);  // half-words 0..7
  for (int k = 0; k < 2; ++k) s += (int64_t)(b[k] & 0xFFFFu) + (int64_t)(b[k] >> 16);  // half-words 8..11
  return (float)(s - 393210) * (1.0f / 65536.0f);
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------------------------------
// Plain-data descriptions shared with the Python side of the tests (ctypes mirrors these).
// ---------------------------------------------------------------------------------------------------
struct oracle_dims {
  int32_t n_envs;         // E: total number of environments of the job (keys the episode ids and slots)
  int32_t n_agents;       // n
  int32_t obs_dim;        // D
  int32_t n_actions;      // A
  int32_t hidden;         // H
  int32_t ring_episodes;  // C, a multiple of E
  int32_t ring_steps;     // L
  int32_t precision;      // 0 = fp32, 1 = bf16 weights and operands
  uint64_t seed;          // key of the epsilon stream
  // Heterogeneous teams (Table I lists a scenario whose team mixes two unit types; Sec. IV discusses it): each
  // unit type may have a network of its own instead of the one shared network.  n_types <= 1 or a null
  // agent_type: one network for every agent.  Otherwise agent i is decided for by network agent_type[i], and
  // every routine below that takes `const oracle_weights* w` is given an array of n_types networks.
  int32_t n_types;
  int32_t reserved;
  const int32_t* agent_type;  // [n], each in [0, n_types)
};

// Seeded synthetic environment standing in for the simulator of Algorithm 1 (Env.step / Env.done).
// All thresholds are 24-bit integers compared with the top 24 bits of a Philox word.
struct oracle_env {
  uint64_t seed;
  int32_t obs_law;              // 0: uniform [-1,1);  1: Irwin-Hall(12) "normal", clipped to [-3,3]
  uint32_t done_thresh24;       // episode ends iff (w >> 8) < done_thresh24
  uint32_t avail_thresh_first;  // actions 1 .. avail_split-1
  uint32_t avail_thresh_rest;   // actions avail_split .. A-1 ; action 0 is always available
  int32_t avail_split;
  int32_t n_type0;              // agents [0, n_type0) are unit type 0, the rest type 1
  int32_t type_block_start;     // obs dims [start, start+len) belong to type 0,
  int32_t type_block_len;       //          [start+len, start+2 len) to type 1; 0 = no typed blocks
};

struct oracle_weights {
  const float* W1;    // [H][D+n+A]
  const float* b1;    // [H]
  const float* W_ih;  // [3H][H]  rows r | z | n
  const float* b_ih;  // [3H]
  const float* W_hh;  // [3H][H]
  const float* b_hh;  // [3H]
  const float* W2;    // [A][H]
  const float* b2;    // [A]
};

// Per-listed-environment recurrent state (Es = number of listed environments).
struct oracle_state {
  float* h;              // [Es][n][H]
  int32_t* last_action;  // [Es][n], -1 = none (episode start)
  int32_t* slot;         // [Es] global ring slot of the open episode
  int32_t* pos;          // [Es] next write position inside the slot
  int64_t* ep_count;     // [Es] episodes this environment has closed
};

// Replay-pool image for the listed environments: S = C/E slots each, local slot index ls = 0..S-1.
struct oracle_ring {
  float* obs;         // [Es*S][L][n][D]
  uint8_t* avail;     // [Es*S][L][n][A]
  int32_t* action;    // [Es*S][L][n]
  float* q;           // [Es*S][L][n][A]
  float* reward;      // [Es*S][L]
  uint8_t* done;      // [Es*S][L]
  int64_t* slot_epid;     // [Es*S], -1 = never used
  int32_t* slot_len;      // [Es*S]
  uint8_t* slot_complete; // [Es*S]
};

// Optional per-step traces (any pointer may be null).
struct oracle_trace {
  float* obs;            // [T][Es][n][D]
  uint8_t* avail;        // [T][Es][n][A]
  float* reward;         // [T][Es]
  uint8_t* done;         // [T][Es]
  float* q;              // [T][Es][n][A]
  float* h;              // [T][Es][n][H]  hidden state after the step, before any reset
  int32_t* action;       // [T][Es][n]  action taken (after adoption, see oracle_rollout)
  int32_t* action_free;  // [T][Es][n]  the oracle's own choice
  uint8_t* explore;      // [T][Es][n]
  float* u;              // [T][Es][n]
  int32_t* slot;         // [T][Es] slot written
  int32_t* pos;          // [T][Es] position written
};

enum { ORACLE_CNT_STEPS = 0, ORACLE_CNT_EPISODES, ORACLE_CNT_EXPLORE, ORACLE_CNT_NO_AVAIL,
       ORACLE_CNT_TRUNCATED, ORACLE_CNT_N };

void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

float oracle_bf16_round(float x) { return bf16_round(x); }

float oracle_uniform24(uint32_t w) { return uniform24(w); }

// Linear epsilon schedule: eps_t = s + (e - s) * min(t, N) / N in double, then rounded to float.
// N <= 0 means "no annealing": eps_t = s.
float oracle_eps_at(double eps_start, double eps_end, int32_t anneal_steps, uint32_t t) {
  if (anneal_steps <= 0) return (float)eps_start;
  const double N = (double)anneal_steps;
  const double tt = (double)t < N ? (double)t : N;
  const double frac = tt / N;
  const double delta = (eps_end - eps_start) * frac;
  return (float)(eps_start + delta);
}

// ---------------------------------------------------------------------------------------------------
// Synthetic environment, one (step, env): observation, availability mask, reward, done.
// ---------------------------------------------------------------------------------------------------
void oracle_env_emit(const oracle_dims* d, const oracle_env* env, uint32_t t, uint32_t e,
                     float* obs /*[n][D]*/, uint8_t* avail /*[n][A]*/, float* reward, uint8_t* done) {
  uint32_t w[4], w2[4];
  // done: block 0 of the (t, e) done/reward stream, word 0
  philox_block(env->seed, t, e, 0, 0, TAG_DONE_REWARD, w);
  *done = ((w[0] >> 8) < env->done_thresh24) ? 1 : 0;
  // reward: blocks 1 and 2
  philox_block(env->seed, t, e, 0, 1, TAG_DONE_REWARD, w);
  philox_block(env->seed, t, e, 0, 2, TAG_DONE_REWARD, w2);
  *reward = irwin_hall12(w, w2);

  for (int i = 0; i < d->n_agents; ++i) {
    for (int a = 0; a < d->n_actions; ++a) {
      uint8_t v = 1;
      if (a > 0) {
        philox_block(env->seed, t, e, (uint32_t)i, (uint32_t)(a / 4), TAG_AVAIL, w);
        const uint32_t thr = (a < env->avail_split) ? env->avail_thresh_first : env->avail_thresh_rest;
        v = ((w[a % 4] >> 8) < thr) ? 1 : 0;
      }
      avail[i * d->n_actions + a] = v;
    }
    const int type = (i < env->n_type0) ? 0 : 1;
    for (int k = 0; k < d->obs_dim; ++k) {
      float v;
      if (env->obs_law == 0) {
        philox_block(env->seed, t, e, (uint32_t)i, (uint32_t)(k / 4), TAG_OBS, w);
        v = (float)((int32_t)(w[k % 4] >> 8) - 8388608) * (1.0f / 8388608.0f);
      } else {
        philox_block(env->seed, t, e, (uint32_t)i, (uint32_t)(2 * k), TAG_OBS, w);
        philox_block(env->seed, t, e, (uint32_t)i, (uint32_t)(2 * k + 1), TAG_OBS, w2);
        v = irwin_hall12(w, w2);
        if (v > 3.0f) v = 3.0f;
        if (v < -3.0f) v = -3.0f;
      }
      if (env->type_block_len > 0) {
        const int other_lo = env->type_block_start + (type == 0 ? env->type_block_len : 0);
        if (k >= other_lo && k < other_lo + env->type_block_len) v = 0.0f;  // the other type's block
      }
      obs[i * d->obs_dim + k] = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// Agent network, one row.  h_prev and the outputs are float (the stored precision).
// ---------------------------------------------------------------------------------------------------
void oracle_agent_forward(const oracle_dims* d, const oracle_weights* w, const float* obs /*[D]*/,
                          int32_t agent, int32_t last_action, const float* h_prev /*[H]*/,
                          float* q_out /*[A]*/, float* h_out /*[H]*/) {
  const int D = d->obs_dim, n = d->n_agents, A = d->n_actions, H = d->hidden;
  const int I = D + n + A;
  const bool lowp = d->precision == 1;
  auto wq = [lowp](float v) { return lowp ? (double)bf16_round(v) : (double)v; };  // matrix entry
  auto op = [lowp](float v) { return lowp ? (double)bf16_round(v) : (double)v; };  // matmul operand

  // fc1 + ReLU.  The one-hot parts of x select one column each.
  std::vector<float> y(H);
  for (int j = 0; j < H; ++j) {
    double acc = (double)w->b1[j];
    for (int k = 0; k < D; ++k) acc += wq(w->W1[j * I + k]) * op(obs[k]);
    acc += wq(w->W1[j * I + D + agent]);
    if (last_action >= 0) acc += wq(w->W1[j * I + D + n + last_action]);
    y[j] = (float)(acc > 0.0 ? acc : 0.0);
  }
  // GRU cell
  std::vector<float> hn(H);
  for (int j = 0; j < H; ++j) {
    double gi[3], gh[3];
    for (int g = 0; g < 3; ++g) {
      const int row = g * H + j;
      double a = (double)w->b_ih[row];
      for (int k = 0; k < H; ++k) a += wq(w->W_ih[row * H + k]) * op(y[k]);
      double b = (double)w->b_hh[row];
      for (int k = 0; k < H; ++k) b += wq(w->W_hh[row * H + k]) * op(h_prev[k]);
      gi[g] = a;
      gh[g] = b;
    }
    const double r = 1.0 / (1.0 + std::exp(-(gi[0] + gh[0])));
    const double z = 1.0 / (1.0 + std::exp(-(gi[1] + gh[1])));
    const double c = std::tanh(gi[2] + r * gh[2]);
    hn[j] = (float)((1.0 - z) * c + z * (double)h_prev[j]);
  }
  // fc2
  for (int a = 0; a < A; ++a) {
    double acc = (double)w->b2[a];
    for (int k = 0; k < H; ++k) acc += wq(w->W2[a * H + k]) * op(hn[k]);
    q_out[a] = (float)acc;
  }
  for (int j = 0; j < H; ++j) h_out[j] = hn[j];
}

// ---------------------------------------------------------------------------------------------------
// Masked greedy choice with the lowest-index tie rule, then the epsilon draw.
//   m = max of Q over available actions (float compares);  thr = m - 1e-4f (one float subtraction);
//   greedy = lowest available a with Q[a] >= thr (lowest available a if no compare succeeds, which
//   only happens with NaN).  Philox block (t, e, i, tag 0): word 0 -> u; explore iff u < eps;
//   word 1 -> index among the K available actions, floor(w1 * K / 2^32), ascending order.
//   A row with no available action takes action 0 and reports it.
// Returns the action; *explore, *u, *no_avail are outputs.
// ---------------------------------------------------------------------------------------------------
int32_t oracle_select_action(const float* q, const uint8_t* avail, int32_t A, float eps, uint64_t seed,
                             uint32_t t, uint32_t e, uint32_t i, uint8_t* explore, float* u_out,
                             uint8_t* no_avail) {
  uint32_t w[4];
  philox_block(seed, t, e, i, 0, TAG_EPS, w);
  const float u = uniform24(w[0]);
  if (u_out) *u_out = u;
  int K = 0;
  for (int a = 0; a < A; ++a) K += avail[a] ? 1 : 0;
  if (no_avail) *no_avail = (K == 0);
  if (K == 0) {
    if (explore) *explore = 0;
    return 0;
  }
  const bool ex = u < eps;
  if (explore) *explore = ex ? 1 : 0;
  if (ex) {
    const uint32_t j = (uint32_t)(((uint64_t)w[1] * (uint64_t)K) >> 32);
    uint32_t seen = 0;
    for (int a = 0; a < A; ++a)
      if (avail[a]) {
        if (seen == j) return a;
        ++seen;
      }
  }
  float m = -INFINITY;
  for (int a = 0; a < A; ++a)
    if (avail[a] && q[a] > m) m = q[a];
  const float thr = m - 1e-4f;
  int first_avail = -1;
  for (int a = 0; a < A; ++a) {
    if (!avail[a]) continue;
    if (first_avail < 0) first_avail = a;
    if (q[a] >= thr) return a;
  }
  return first_avail;
}

// The same choice for N independent rows (a plain loop over oracle_select_action).
//   q [N][A], avail [N][A], eps [N], t/e/i [N]  ->  action [N], explore [N]
void oracle_select_batch(const float* q, const uint8_t* avail, int32_t A, int64_t N, const float* eps,
                         uint64_t seed, const uint32_t* t, const uint32_t* e, const uint32_t* i,
                         int32_t* action, uint8_t* explore) {
  for (int64_t r = 0; r < N; ++r) {
    uint8_t ex = 0;
    action[r] = oracle_select_action(q + r * A, avail + r * A, A, eps[r], seed, t[r], e[r], i[r], &ex,
                                     nullptr, nullptr);
    if (explore) explore[r] = ex;
  }
}

// ---------------------------------------------------------------------------------------------------
// State and ring initialisation for a list of environments.
// ---------------------------------------------------------------------------------------------------
void oracle_init(const oracle_dims* d, const int32_t* env_ids, int32_t Es, oracle_state* st,
                 oracle_ring* ring) {
  const int S = d->ring_episodes / d->n_envs;
  for (int x = 0; x < Es; ++x) {
    for (int k = 0; k < d->n_agents * d->hidden; ++k) st->h[(size_t)x * d->n_agents * d->hidden + k] = 0.0f;
    for (int i = 0; i < d->n_agents; ++i) st->last_action[x * d->n_agents + i] = -1;
    st->slot[x] = env_ids[x] * S;
    st->pos[x] = 0;
    st->ep_count[x] = 0;
    if (ring) {
      for (int ls = 0; ls < S; ++ls) {
        ring->slot_epid[x * S + ls] = -1;
        ring->slot_len[x * S + ls] = 0;
        ring->slot_complete[x * S + ls] = 0;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// One decision step for the listed environments, given what the environments sent (Algorithm 2 body:
// get observations, decide, send actions) plus the recording of the step and the episode bookkeeping of
// Algorithm 1 (record each step; at the end of the game hand the track over and reset).
//
//   obs [Es][n][D], avail [Es][n][A], reward [Es], done [Es] : this step's environment outputs
//   adopt [Es][n] or null: if given and adopt != the oracle's own choice, the adopted action is the
//       one recorded and fed back as "last action" (used by the parity referee to stay in lock-step
//       with another implementation across numerical near-ties); the own choice is still traced.
//   tr / tstep: optional trace, written at step index tstep of a trace holding Es rows per step.
// ---------------------------------------------------------------------------------------------------
// The network that decides for agent i: the shared one, or the one of the agent's unit type.
static const oracle_weights* network_of(const oracle_dims* d, const oracle_weights* w, int agent) {
  if (d->n_types <= 1 || d->agent_type == nullptr) return w;
  return w + d->agent_type[agent];
}

static void step_range(const oracle_dims* d, const oracle_weights* w, const int32_t* env_ids, int x0,
                       int x1, int32_t Es, uint32_t t, float eps, const float* obs,
                       const uint8_t* avail, const float* reward, const uint8_t* done,
                       const int32_t* adopt, oracle_state* st, oracle_ring* ring, int32_t* actions_out,
                       oracle_trace* tr, int32_t tstep, uint64_t* counters) {
  const int n = d->n_agents, D = d->obs_dim, A = d->n_actions, H = d->hidden, L = d->ring_steps;
  const int E = d->n_envs;
  const int S = d->ring_episodes / E;
  std::vector<float> q(A), hnew((size_t)n * H);
  for (int x = x0; x < x1; ++x) {
    const int e = env_ids[x];
    const int slot = st->slot[x], pos = st->pos[x];
    const int ls = slot - e * S;                       // local slot index inside this env's sub-ring
    const size_t rs = (size_t)x * S + ls;              // row of the ring image
    if (ring && pos == 0) {                            // an episode opens in this slot
      ring->slot_epid[rs] = st->ep_count[x] * (int64_t)E + e;
      ring->slot_len[rs] = 0;
      ring->slot_complete[rs] = 0;
    }
    for (int i = 0; i < n; ++i) {
      const size_t row = (size_t)x * n + i;
      const float* o = obs + row * D;
      const uint8_t* av = avail + row * A;
      float* hp = st->h + row * H;
      oracle_agent_forward(d, network_of(d, w, i), o, i, st->last_action[row], hp, q.data(),
                           hnew.data() + (size_t)i * H);
      uint8_t ex = 0, na = 0;
      float u = 0.f;
      const int32_t a_free = oracle_select_action(q.data(), av, A, eps, d->seed, t, (uint32_t)e,
                                                  (uint32_t)i, &ex, &u, &na);
      const int32_t a_used = adopt ? adopt[row] : a_free;
      counters[ORACLE_CNT_STEPS] += 1;
      counters[ORACLE_CNT_EXPLORE] += ex;
      counters[ORACLE_CNT_NO_AVAIL] += na;
      if (actions_out) actions_out[row] = a_used;
      if (ring) {
        const size_t rr = (rs * L + pos) * n + i;
        std::memcpy(ring->obs + rr * D, o, sizeof(float) * D);
        std::memcpy(ring->avail + rr * A, av, A);
        std::memcpy(ring->q + rr * A, q.data(), sizeof(float) * A);
        ring->action[rr] = a_used;
      }
      if (tr) {
        const size_t trow = ((size_t)tstep * Es + x) * n + i;
        if (tr->obs) std::memcpy(tr->obs + trow * D, o, sizeof(float) * D);
        if (tr->avail) std::memcpy(tr->avail + trow * A, av, A);
        if (tr->q) std::memcpy(tr->q + trow * A, q.data(), sizeof(float) * A);
        if (tr->h) std::memcpy(tr->h + trow * H, hnew.data() + (size_t)i * H, sizeof(float) * H);
        if (tr->action) tr->action[trow] = a_used;
        if (tr->action_free) tr->action_free[trow] = a_free;
        if (tr->explore) tr->explore[trow] = ex;
        if (tr->u) tr->u[trow] = u;
      }
      st->last_action[row] = a_used;
    }
    if (ring) {
      ring->reward[rs * L + pos] = reward[x];
      ring->done[rs * L + pos] = done[x];
      ring->slot_len[rs] = pos + 1;
    }
    if (tr) {
      const size_t te = (size_t)tstep * Es + x;
      if (tr->reward) tr->reward[te] = reward[x];
      if (tr->done) tr->done[te] = done[x];
      if (tr->slot) tr->slot[te] = slot;
      if (tr->pos) tr->pos[te] = pos;
    }
    const bool ended = done[x] != 0;
    const bool full = (pos + 1 == L);
    if (ended || full) {
      // the episode closes: whole track is complete; fresh hidden state and no last action
      if (ring) ring->slot_complete[rs] = 1;
      counters[ORACLE_CNT_EPISODES] += 1;
      if (!ended) counters[ORACLE_CNT_TRUNCATED] += 1;
      st->ep_count[x] += 1;
      st->slot[x] = e * S + (int)(st->ep_count[x] % S);
      st->pos[x] = 0;
      for (int k = 0; k < n * H; ++k) st->h[(size_t)x * n * H + k] = 0.0f;
      for (int i = 0; i < n; ++i) st->last_action[x * n + i] = -1;
    } else {
      st->pos[x] = pos + 1;
      std::memcpy(st->h + (size_t)x * n * H, hnew.data(), sizeof(float) * (size_t)n * H);
    }
  }
}

}  // extern "C" (reopened below)

namespace {
// Environments are independent, so a step may be split over threads by environment range.
void parallel_over_envs(int Es, int n_threads, uint64_t* counters,
                        const std::function<void(int, int, uint64_t*)>& body) {
  if (n_threads < 1) n_threads = 1;
  if (n_threads > Es) n_threads = Es > 0 ? Es : 1;
  std::vector<std::vector<uint64_t>> local(n_threads, std::vector<uint64_t>(ORACLE_CNT_N, 0));
  if (n_threads == 1) {
    body(0, Es, local[0].data());
  } else {
    std::vector<std::thread> th;
    for (int k = 0; k < n_threads; ++k) {
      const int x0 = (int)((int64_t)Es * k / n_threads), x1 = (int)((int64_t)Es * (k + 1) / n_threads);
      th.emplace_back([&, k, x0, x1] { body(x0, x1, local[k].data()); });
    }
    for (auto& t : th) t.join();
  }
  for (int k = 0; k < n_threads; ++k)
    for (int c = 0; c < ORACLE_CNT_N; ++c) counters[c] += local[k][c];
}
}  // namespace

extern "C" {

void oracle_step(const oracle_dims* d, const oracle_weights* w, const int32_t* env_ids, int32_t Es,
                 uint32_t t, float eps, const float* obs, const uint8_t* avail, const float* reward,
                 const uint8_t* done, const int32_t* adopt, oracle_state* st, oracle_ring* ring,
                 int32_t* actions_out, oracle_trace* tr, int32_t tstep, uint64_t* counters,
                 int32_t n_threads) {
  parallel_over_envs(Es, n_threads, counters, [&](int x0, int x1, uint64_t* cnt) {
    step_range(d, w, env_ids, x0, x1, Es, t, eps, obs, avail, reward, done, adopt, st, ring,
               actions_out, tr, tstep, cnt);
  });
}

// ---------------------------------------------------------------------------------------------------
// The same step when the environment answers after the action (Algorithm 1: the actor sends its observation,
// receives the action and only then steps the environment): the reward and the end-of-game flag of an action reach the worker with the NEXT
// observation of that environment.  For each listed environment, in this order:
//   1. if a record of the open episode is still waiting for its outcome (pos > 0): prev_reward / prev_done
//      are written into that record (pos - 1); if the game ended, or the slot is full (pos == L), the
//      episode closes exactly as in the synchronous step (header, counters, next slot, zero hidden state,
//      no last action);
//   2. the decision on this observation, recorded at (slot, pos) with reward 0 and done 0 for now;
//      the cursor moves on and the slot's length counts the new record.
// An environment's first call has nothing waiting, so its prev_reward / prev_done are ignored.
// ---------------------------------------------------------------------------------------------------
void oracle_step_lagged(const oracle_dims* d, const oracle_weights* w, const int32_t* env_ids, int32_t Es,
                        uint32_t t, float eps, const float* obs, const uint8_t* avail,
                        const float* prev_reward, const uint8_t* prev_done, const int32_t* adopt,
                        oracle_state* st, oracle_ring* ring, int32_t* actions_out, oracle_trace* tr,
                        uint64_t* counters) {
  const int n = d->n_agents, D = d->obs_dim, A = d->n_actions, H = d->hidden, L = d->ring_steps;
  const int E = d->n_envs;
  const int S = d->ring_episodes / E;
  std::vector<float> q(A), hnew((size_t)n * H);
  for (int x = 0; x < Es; ++x) {
    const int e = env_ids[x];
    // ---- 1. the outcome of the previous action ----
    if (st->pos[x] > 0) {
      const int pos = st->pos[x];
      const size_t rs = (size_t)x * S + (st->slot[x] - e * S);
      if (ring) {
        ring->reward[rs * L + pos - 1] = prev_reward[x];
        ring->done[rs * L + pos - 1] = prev_done[x];
      }
      const bool ended = prev_done[x] != 0;
      if (ended || pos == L) {
        if (ring) ring->slot_complete[rs] = 1;
        counters[ORACLE_CNT_EPISODES] += 1;
        if (!ended) counters[ORACLE_CNT_TRUNCATED] += 1;
        st->ep_count[x] += 1;
        st->slot[x] = e * S + (int)(st->ep_count[x] % S);
        st->pos[x] = 0;
        for (int k = 0; k < n * H; ++k) st->h[(size_t)x * n * H + k] = 0.0f;
        for (int i = 0; i < n; ++i) st->last_action[x * n + i] = -1;
      }
    }
    // ---- 2. the decision on this observation ----
    const int slot = st->slot[x], pos = st->pos[x];
    const size_t rs = (size_t)x * S + (slot - e * S);
    if (ring && pos == 0) {
      ring->slot_epid[rs] = st->ep_count[x] * (int64_t)E + e;
      ring->slot_len[rs] = 0;
      ring->slot_complete[rs] = 0;
    }
    for (int i = 0; i < n; ++i) {
      const size_t row = (size_t)x * n + i;
      const float* o = obs + row * D;
      const uint8_t* av = avail + row * A;
      oracle_agent_forward(d, network_of(d, w, i), o, i, st->last_action[row], st->h + row * H, q.data(),
                           hnew.data() + (size_t)i * H);
      uint8_t ex = 0, na = 0;
      float u = 0.f;
      const int32_t a_free = oracle_select_action(q.data(), av, A, eps, d->seed, t, (uint32_t)e,
                                                  (uint32_t)i, &ex, &u, &na);
      const int32_t a_used = adopt ? adopt[row] : a_free;
      counters[ORACLE_CNT_STEPS] += 1;
      counters[ORACLE_CNT_EXPLORE] += ex;
      counters[ORACLE_CNT_NO_AVAIL] += na;
      if (actions_out) actions_out[row] = a_used;
      if (ring) {
        const size_t rr = (rs * L + pos) * n + i;
        std::memcpy(ring->obs + rr * D, o, sizeof(float) * D);
        std::memcpy(ring->avail + rr * A, av, A);
        std::memcpy(ring->q + rr * A, q.data(), sizeof(float) * A);
        ring->action[rr] = a_used;
      }
      if (tr) {
        const size_t trow = (size_t)x * n + i;
        if (tr->q) std::memcpy(tr->q + trow * A, q.data(), sizeof(float) * A);
        if (tr->action_free) tr->action_free[trow] = a_free;
        if (tr->explore) tr->explore[trow] = ex;
      }
      st->last_action[row] = a_used;
    }
    if (ring) {
      ring->reward[rs * L + pos] = 0.0f;
      ring->done[rs * L + pos] = 0;
      ring->slot_len[rs] = pos + 1;
    }
    st->pos[x] = pos + 1;
    std::memcpy(st->h + (size_t)x * n * H, hnew.data(), sizeof(float) * (size_t)n * H);
  }
}

// ---------------------------------------------------------------------------------------------------
// T steps against the synthetic environment, starting at global step t0.
//   adopt [T][Es][n] or null (see oracle_step).  eps follows oracle_eps_at with the global step index.
// Each thread owns a range of environments and walks its own steps; the result does not depend on
// the number of threads.
// ---------------------------------------------------------------------------------------------------
void oracle_rollout(const oracle_dims* d, const oracle_weights* w, const oracle_env* env,
                    const int32_t* env_ids, int32_t Es, uint32_t t0, int32_t T, double eps_start,
                    double eps_end, int32_t anneal_steps, const int32_t* adopt, oracle_state* st,
                    oracle_ring* ring, oracle_trace* tr, uint64_t* counters, int32_t n_threads) {
  const int n = d->n_agents, D = d->obs_dim, A = d->n_actions;
  parallel_over_envs(Es, n_threads, counters, [&](int x0, int x1, uint64_t* cnt) {
    std::vector<float> obs((size_t)Es * n * D);   // indexed by x like the caller's arrays
    std::vector<uint8_t> avail((size_t)Es * n * A);
    std::vector<float> reward(Es);
    std::vector<uint8_t> done(Es);
    for (int s = 0; s < T; ++s) {
      const uint32_t t = t0 + (uint32_t)s;
      const float eps = oracle_eps_at(eps_start, eps_end, anneal_steps, t);
      for (int x = x0; x < x1; ++x)
        oracle_env_emit(d, env, t, (uint32_t)env_ids[x], obs.data() + (size_t)x * n * D,
                        avail.data() + (size_t)x * n * A, &reward[x], &done[x]);
      step_range(d, w, env_ids, x0, x1, Es, t, eps, obs.data(), avail.data(), reward.data(),
                 done.data(), adopt ? adopt + (size_t)s * Es * n : nullptr, st, ring, nullptr, tr, s,
                 cnt);
    }
  });
}

// Host cores this process may run on.
int32_t oracle_hardware_threads(void) {
  cpu_set_t set;
  CPU_ZERO(&set);
  if (sched_getaffinity(0, sizeof(set), &set) == 0) {
    const int c = CPU_COUNT(&set);
    if (c > 0) return c;
  }
  const unsigned c = std::thread::hardware_concurrency();
  return c ? (int32_t)c : 1;
}

}  // extern "C"
