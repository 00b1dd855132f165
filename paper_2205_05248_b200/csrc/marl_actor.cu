// Host runtime and C ABI of the actor library: configuration checks, buffer carving, weight repacking,
// launch planning and the entry points declared in include/marl_actor.h.  All arithmetic of the actor
// step runs in the kernels (actor_ffma.cu, actor_tc.cu, env_kernel.cu); nothing here computes on the CPU
// and there is no CPU fallback.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"

namespace marl {
int launch_env_generate(const marl_synth_env_t& env, int E, int n, int D, int A, uint32_t t0, int n_steps,
                        float* obs, uint8_t* avail, float* reward, uint8_t* done, int sms, cudaStream_t stream);
void ffma_tiling(int E, int n, int sms, int* ept, int* num_tiles);
size_t ffma_smem_bytes(int n, int D, int A, int H);
int launch_actor_ffma(const ActorParams& p, int sms, cudaStream_t stream);
// tensor-core kernel
bool tc_supported(int n, int D, int A, int H, int prec);
size_t tc_wpack_bytes(int n, int D, int A, int H);
void tc_pack_weights(int n, int D, int A, int H, const float* W1, const float* b1, const float* Wih,
                     const float* bih, const float* Whh, const float* bhh, const float* W2, const float* b2,
                     void* dst_host);
void tc_tiling(int E, int n, int sms, int* ept, int* num_tiles);
int launch_actor_tc(const ActorParams& p, int sms, cudaStream_t stream);
bool tcp_supported(int n, int D, int A, int H, int prec);
int launch_actor_tcp(const ActorParams& p, int sms, cudaStream_t stream);
bool tc2_supported(int n, int D, int A, int H, int prec);
int launch_actor_tc2(const ActorParams& p, int sms, cudaStream_t stream);
bool tcw_supported(int n, int D, int A, int H, int prec);
int launch_actor_tcw(const ActorParams& p, int sms, cudaStream_t stream);
int launch_ring_sample(const SampleParams& p, cudaStream_t stream);
}  // namespace marl

using namespace marl;

static thread_local std::string g_err;

static int fail(int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}

#define CU_TRY(call)                                                                              \
  do {                                                                                            \
    const cudaError_t e_ = (call);                                                                \
    if (e_ != cudaSuccess) return fail(MARL_ECUDA, "%s: %s", #call, cudaGetErrorString(e_));      \
  } while (0)

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Carve {
  size_t off = 0;
  size_t take(size_t bytes) {
    const size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  }
};

struct FfmaWeightOffsets { size_t W1T, b1, WihT, bih, WhhT, bhh, W2, b2, total; };

static FfmaWeightOffsets ffma_weight_offsets(int n, int D, int A, int H) {
  const int I = D + n + A;
  FfmaWeightOffsets w;
  Carve c;
  w.W1T = c.take(sizeof(float) * (size_t)(I + 4) * H);
  w.b1 = c.take(sizeof(float) * H);
  w.WihT = c.take(sizeof(float) * (size_t)H * 3 * H);
  w.bih = c.take(sizeof(float) * 3 * H);
  w.WhhT = c.take(sizeof(float) * (size_t)H * 3 * H);
  w.bhh = c.take(sizeof(float) * 3 * H);
  w.W2 = c.take(sizeof(float) * (size_t)A * H);
  w.b2 = c.take(sizeof(float) * 32);
  w.total = c.off;
  return w;
}

struct StateOffsets { size_t h, last_action, slot, pos, ep_count, counters, status, wff[2], wpack[2], ids, total; };  // two weight images
struct RingOffsets { size_t records, epid, len, complete, total; };
struct WorkOffsets { size_t obs, avail, reward, done, actions, total; };

static RecordLayout record_layout(int n, int D, int A) {
  RecordLayout r;
  size_t o = 0;
  r.off_obs = (uint32_t)o; o = align_up(o + sizeof(float) * n * D, 16);
  r.off_avail = (uint32_t)o; o = align_up(o + (size_t)n * A, 16);
  r.off_action = (uint32_t)o; o = align_up(o + sizeof(int32_t) * n, 16);
  r.off_q = (uint32_t)o; o = align_up(o + sizeof(float) * n * A, 16);
  r.off_reward = (uint32_t)o;
  r.off_done = (uint32_t)o + 4;
  o += 16;
  r.rec_bytes = (uint32_t)o;
  r.pad = 0;
  return r;
}

static StateOffsets state_offsets(const marl_actor_config_t& c) {
  StateOffsets s;
  Carve cv;
  const size_t rows = (size_t)c.n_envs * c.n_agents;
  s.h = cv.take(sizeof(float) * rows * c.hidden);
  s.last_action = cv.take(sizeof(int32_t) * rows);
  s.slot = cv.take(sizeof(int32_t) * c.n_envs);
  s.pos = cv.take(sizeof(int32_t) * c.n_envs);
  s.ep_count = cv.take(sizeof(int64_t) * c.n_envs);
  s.counters = cv.take(sizeof(uint64_t) * CNT_N);
  s.status = cv.take(sizeof(uint32_t) * 4);
  const size_t types = c.n_agent_types > 1 ? (size_t)c.n_agent_types : 1;  // FFMA images of a typed actor, one per type
  for (int i = 0; i < 2; ++i) {
    s.wff[i] = cv.take(types * ffma_weight_offsets(c.n_agents, c.obs_dim, c.n_actions, c.hidden).total);
    s.wpack[i] = cv.take(tc_wpack_bytes(c.n_agents, c.obs_dim, c.n_actions, c.hidden));
  }
  s.ids = cv.take(sizeof(int32_t) * (size_t)c.n_envs);  // environment list of a partial step
  s.total = cv.off;
  return s;
}

static RingOffsets ring_offsets(const marl_actor_config_t& c) {
  RingOffsets r;
  Carve cv;
  const RecordLayout rl = record_layout(c.n_agents, c.obs_dim, c.n_actions);
  r.records = cv.take((size_t)c.ring_episodes * c.ring_steps * rl.rec_bytes);
  r.epid = cv.take(sizeof(int64_t) * c.ring_episodes);
  r.len = cv.take(sizeof(int32_t) * c.ring_episodes);
  r.complete = cv.take((size_t)c.ring_episodes);
  r.total = cv.off;
  return r;
}

// Staging of W steps of environment output plus one step of actions.
static WorkOffsets work_offsets(const marl_actor_config_t& c, size_t W) {
  WorkOffsets w;
  Carve cv;
  const size_t rows = (size_t)c.n_envs * c.n_agents;
  w.obs = cv.take(sizeof(float) * rows * c.obs_dim * W);
  w.avail = cv.take(rows * c.n_actions * W);
  w.reward = cv.take(sizeof(float) * c.n_envs * W);
  w.done = cv.take((size_t)c.n_envs * W);
  w.actions = cv.take(sizeof(int32_t) * rows);
  w.total = cv.off;
  return w;
}

static int check_config(const marl_actor_config_t* c) {
  if (!c) return fail(MARL_EINVAL, "config is NULL");
  if (c->n_envs < 1) return fail(MARL_EINVAL, "n_envs must be >= 1");
  if (c->n_agents < 1 || c->n_agents > 32) return fail(MARL_EINVAL, "n_agents must be in [1, 32]");
  if (c->obs_dim < 1 || c->obs_dim > 512) return fail(MARL_EINVAL, "obs_dim must be in [1, 512]");
  if (c->n_actions < 1 || c->n_actions > 32) return fail(MARL_EINVAL, "n_actions must be in [1, 32]");
  if (c->hidden != 64 && c->hidden != 128) return fail(MARL_EINVAL, "hidden must be 64 or 128");
  if (c->ring_steps < 1) return fail(MARL_EINVAL, "ring_steps must be >= 1");
  if (c->ring_episodes < c->n_envs || c->ring_episodes % c->n_envs != 0)
    return fail(MARL_EINVAL, "ring_episodes must be a positive multiple of n_envs");
  if (c->precision != MARL_PRECISION_FP32 && c->precision != MARL_PRECISION_BF16)
    return fail(MARL_EINVAL, "unknown precision");
  if (c->kernel < MARL_KERNEL_AUTO || c->kernel > MARL_KERNEL_TENSOR_DUAL) return fail(MARL_EINVAL, "unknown kernel");
  if (c->n_agent_types < 0 || c->n_agent_types > MARL_MAX_AGENT_TYPES)
    return fail(MARL_EINVAL, "n_agent_types must be in [0, %d]", MARL_MAX_AGENT_TYPES);
  if ((double)c->n_envs * c->n_agents > 1.0e9) return fail(MARL_EINVAL, "n_envs * n_agents too large");
  return MARL_OK;
}

struct marl_actor {
  marl_actor_config_t cfg;
  cudaStream_t stream;
  int device, sms;
  bool use_tc;   // a tensor-core kernel steps this actor
  bool use_tcp;  // ... the pipelined one (falls back to the one-tile kernel for inputs it cannot bulk-copy)
  bool use_tc2;  // ... with two tiles resident per SM where a launch allows it (else the pipelined kernel, same results)
  bool tc_allowed, tcp_allowed, tc2_allowed;  // the choice made at creation; per-type networks switch the tensor-core kernels off
  int32_t n_types;               // > 1: per-type networks are loaded
  uint64_t agent_type_bits;
  uint8_t *ring, *state, *work;
  bool own_ring, own_state, own_work;
  size_t work_bytes;
  StateOffsets so;
  RingOffsets ro;
  FfmaWeightOffsets wo;
  RecordLayout rl;
  uint64_t step;
  uint64_t weights_version;
  bool have_weights;
  int32_t* trace_actions;
  float* trace_q;
  int32_t trace_cap, trace_next;
  uint64_t launches;
  std::vector<uint8_t> host_pack;
  // weight publication: the image in use, the copy stream, and the publication waiting for its step
  int wslot;
  cudaStream_t copy_stream;
  cudaEvent_t upload_done, image_free;
  bool image_free_recorded, pending;
  uint64_t pending_version, pending_step;
  std::vector<uint8_t> id_seen;  // scratch of marl_actor_step_subset
  // pinned staging of the environment list, two buffers in turn, each with the event of its last upload
  int32_t* ids_host[2];
  cudaEvent_t ids_copied[2];
  bool ids_in_flight[2];
  int ids_next;
  uint8_t* host_pack2;  // pinned, so that the upload really runs beside the steps
};

__global__ void init_state_kernel(int E, int n, int H, int S, int C, float* h, int32_t* la, int32_t* slot,
                                  int32_t* pos, long long* epc, long long* epid, int32_t* len,
                                  uint8_t* complete, unsigned long long* counters, uint32_t* status) {
  const long long rows = (long long)E * n;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long i0 = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  for (long long i = i0; i < rows * H; i += stride) h[i] = 0.f;
  for (long long i = i0; i < rows; i += stride) la[i] = -1;
  for (long long i = i0; i < E; i += stride) {
    slot[i] = (int32_t)(i * S);
    pos[i] = 0;
    epc[i] = 0;
  }
  for (long long i = i0; i < C; i += stride) {
    epid[i] = -1;
    len[i] = 0;
    complete[i] = 0;
  }
  if (i0 < CNT_N) counters[i0] = 0;
  if (i0 < 4) status[i0] = 0;
}

static int enqueue_reset(marl_actor* a) {
  const marl_actor_config_t& c = a->cfg;
  uint8_t* st = a->state;
  init_state_kernel<<<a->sms * 4, 256, 0, a->stream>>>(
      c.n_envs, c.n_agents, c.hidden, c.ring_episodes / c.n_envs, c.ring_episodes,
      reinterpret_cast<float*>(st + a->so.h), reinterpret_cast<int32_t*>(st + a->so.last_action),
      reinterpret_cast<int32_t*>(st + a->so.slot), reinterpret_cast<int32_t*>(st + a->so.pos),
      reinterpret_cast<long long*>(st + a->so.ep_count), reinterpret_cast<long long*>(a->ring + a->ro.epid),
      reinterpret_cast<int32_t*>(a->ring + a->ro.len), a->ring + a->ro.complete,
      reinterpret_cast<unsigned long long*>(st + a->so.counters), reinterpret_cast<uint32_t*>(st + a->so.status));
  CU_TRY(cudaGetLastError());
  a->launches += 1;
  a->step = 0;
  a->trace_next = 0;
  return MARL_OK;
}

extern "C" {

const char* marl_last_error(void) { return g_err.c_str(); }

int marl_actor_query_sizes(const marl_actor_config_t* cfg, marl_actor_sizes_t* out) {
  const int rc = check_config(cfg);
  if (rc) return rc;
  if (!out) return fail(MARL_EINVAL, "out is NULL");
  out->ring_bytes = ring_offsets(*cfg).total;
  out->state_bytes = state_offsets(*cfg).total;
  out->work_bytes_min = work_offsets(*cfg, 1).total;
  out->work_bytes_per_step = work_offsets(*cfg, 2).total - work_offsets(*cfg, 1).total + 4 * 256;
  return MARL_OK;
}

int marl_actor_create(const marl_actor_config_t* cfg, marl_actor_t** out) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!out) return fail(MARL_EINVAL, "out is NULL");
  *out = nullptr;
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CU_TRY(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10)
    return fail(MARL_ECUDA, "device %s has compute capability %d.%d; this library is built for sm_100a only",
                prop.name, prop.major, prop.minor);
  marl_actor* a = new (std::nothrow) marl_actor();
  if (!a) return fail(MARL_ENOMEM, "out of host memory");
  a->cfg = *cfg;
  a->stream = reinterpret_cast<cudaStream_t>(cfg->stream);
  a->device = dev;
  a->sms = prop.multiProcessorCount;
  a->so = state_offsets(*cfg);
  a->ro = ring_offsets(*cfg);
  a->wo = ffma_weight_offsets(cfg->n_agents, cfg->obs_dim, cfg->n_actions, cfg->hidden);
  a->rl = record_layout(cfg->n_agents, cfg->obs_dim, cfg->n_actions);
  a->ring = a->state = a->work = nullptr;
  a->own_ring = a->own_state = a->own_work = false;
  a->step = 0;
  a->weights_version = 0;
  a->have_weights = false;
  a->trace_actions = nullptr;
  a->trace_q = nullptr;
  a->trace_cap = a->trace_next = 0;
  a->launches = 0;
  a->wslot = 0;
  a->host_pack2 = nullptr;
  a->ids_host[0] = a->ids_host[1] = nullptr;
  a->ids_copied[0] = a->ids_copied[1] = nullptr;
  a->ids_in_flight[0] = a->ids_in_flight[1] = false;
  a->ids_next = 0;
  a->copy_stream = nullptr;
  a->upload_done = a->image_free = nullptr;
  a->image_free_recorded = a->pending = false;
  a->pending_version = a->pending_step = 0;

  const bool tc_ok = tc_supported(cfg->n_agents, cfg->obs_dim, cfg->n_actions, cfg->hidden, cfg->precision);
  const bool tcp_ok = tcp_supported(cfg->n_agents, cfg->obs_dim, cfg->n_actions, cfg->hidden, cfg->precision) ||
                      tcw_supported(cfg->n_agents, cfg->obs_dim, cfg->n_actions, cfg->hidden, cfg->precision);
  const bool tc2_ok = tc2_supported(cfg->n_agents, cfg->obs_dim, cfg->n_actions, cfg->hidden, cfg->precision) && tcp_ok;
  if ((cfg->kernel == MARL_KERNEL_TENSOR && !tc_ok) || (cfg->kernel == MARL_KERNEL_TENSOR_PIPELINED && !tcp_ok) ||
      (cfg->kernel == MARL_KERNEL_TENSOR_DUAL && !tc2_ok)) {
    delete a;
    return fail(MARL_EINVAL, "the tensor-core kernel does not support this shape/precision");
  }
  // Kernel choice.  fp32 precision: the CUDA-core kernel (tensor cores cannot meet its 1e-5 tolerance).  bf16: a
  // tensor-core kernel wherever the shape is supported, at every batch size - timed on the same rollouts from 24
  // rows to 16384 (`bench.py --crossover`), one 128-row tcgen05 tile takes 3.3-5.2 us per
  // environment step against 18-21 us for the CUDA-core kernel's 64-row tiles, so there is no batch size at which
  // the CUDA cores win.
  // (the two-tile kernel is never the automatic choice: measured at workload 5 it is slower than the pipelined kernel -
  // 8.4 ms against 6.15 ms per 64-step rollout - because with the epilogue threads busy all the time the converter
  // warps no longer keep up)
  a->use_tc2 = cfg->kernel == MARL_KERNEL_TENSOR_DUAL;
  a->use_tcp = cfg->kernel == MARL_KERNEL_TENSOR_PIPELINED || a->use_tc2 || (cfg->kernel == MARL_KERNEL_AUTO && tcp_ok);
  a->use_tc = tc_ok && cfg->kernel != MARL_KERNEL_FFMA;
  a->tc2_allowed = a->use_tc2;
  a->tcp_allowed = a->use_tcp;
  a->tc_allowed = a->use_tc;
  a->n_types = 1;
  a->agent_type_bits = 0;

  auto bind = [&](void* mem, size_t have, size_t need, uint8_t** dst, bool* own, const char* what) -> int {
    if (mem) {
      if (reinterpret_cast<uintptr_t>(mem) % 256) return fail(MARL_EALIGN, "%s must be 256-byte aligned", what);
      if (have < need) return fail(MARL_ENOMEM, "%s: %zu bytes given, %zu needed", what, have, need);
      *dst = static_cast<uint8_t*>(mem);
      *own = false;
    } else {
      void* p = nullptr;
      const cudaError_t e = cudaMalloc(&p, need);
      if (e != cudaSuccess) return fail(MARL_ENOMEM, "cudaMalloc(%zu) for %s: %s", need, what, cudaGetErrorString(e));
      *dst = static_cast<uint8_t*>(p);
      *own = true;
    }
    return MARL_OK;
  };
  const size_t work_min = work_offsets(*cfg, 1).total;
  rc = bind(cfg->ring_mem, cfg->ring_bytes, a->ro.total, &a->ring, &a->own_ring, "ring_mem");
  if (!rc) rc = bind(cfg->state_mem, cfg->state_bytes, a->so.total, &a->state, &a->own_state, "state_mem");
  if (!rc) {
    a->work_bytes = cfg->work_mem ? cfg->work_bytes : work_min;
    rc = bind(cfg->work_mem, cfg->work_bytes, work_min, &a->work, &a->own_work, "work_mem");
  }
  if (!rc) rc = enqueue_reset(a);
  if (rc) {
    const std::string keep = g_err;
    if (a->own_ring && a->ring) cudaFree(a->ring);
    if (a->own_state && a->state) cudaFree(a->state);
    if (a->own_work && a->work) cudaFree(a->work);
    delete a;
    g_err = keep;
    return rc;
  }
  *out = a;
  return MARL_OK;
}

void marl_actor_destroy(marl_actor_t* a) {
  if (!a) return;
  cudaStreamSynchronize(a->stream);
  if (a->copy_stream) {
    cudaStreamSynchronize(a->copy_stream);
    cudaStreamDestroy(a->copy_stream);
    cudaEventDestroy(a->upload_done);
    cudaEventDestroy(a->image_free);
    cudaFreeHost(a->host_pack2);
  }
  for (int i = 0; i < 2; ++i) {
    if (a->ids_host[i]) cudaFreeHost(a->ids_host[i]);
    if (a->ids_copied[i]) cudaEventDestroy(a->ids_copied[i]);
  }
  if (a->own_ring) cudaFree(a->ring);
  if (a->own_state) cudaFree(a->state);
  if (a->own_work) cudaFree(a->work);
  delete a;
}

static float to_bf16_value(float v) {
  uint32_t u;
  memcpy(&u, &v, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return v;
  u += 0x7FFFu + ((u >> 16) & 1u);
  u &= 0xFFFF0000u;
  memcpy(&v, &u, 4);
  return v;
}

// Packs the network into `dst` as the kernels read it: the FFMA image (k-major fp32, bf16-representable values in
// the bf16 precision) followed by the tensor-core image.
static void pack_weights_host(marl_actor* a, const float* W1, const float* b1, const float* W_ih, const float* b_ih,
                              const float* W_hh, const float* b_hh, const float* W2, const float* b2,
                              uint8_t* hp) {
  const int n = a->cfg.n_agents, D = a->cfg.obs_dim, A = a->cfg.n_actions, H = a->cfg.hidden;
  const int I = D + n + A;
  const bool lowp = a->cfg.precision == MARL_PRECISION_BF16;
  const size_t tcb = tc_wpack_bytes(n, D, A, H);
  memset(hp, 0, a->wo.total + tcb);
  auto q = [lowp](float v) { return lowp ? to_bf16_value(v) : v; };
  float* W1T = reinterpret_cast<float*>(hp + a->wo.W1T);
  for (int j = 0; j < H; ++j)
    for (int k = 0; k < I; ++k) W1T[(size_t)k * H + j] = q(W1[(size_t)j * I + k]);
  float* WihT = reinterpret_cast<float*>(hp + a->wo.WihT);
  float* WhhT = reinterpret_cast<float*>(hp + a->wo.WhhT);
  for (int r = 0; r < 3 * H; ++r)
    for (int k = 0; k < H; ++k) {
      WihT[(size_t)k * 3 * H + r] = q(W_ih[(size_t)r * H + k]);
      WhhT[(size_t)k * 3 * H + r] = q(W_hh[(size_t)r * H + k]);
    }
  float* W2p = reinterpret_cast<float*>(hp + a->wo.W2);
  for (int i = 0; i < A * H; ++i) W2p[i] = q(W2[i]);
  memcpy(hp + a->wo.b1, b1, sizeof(float) * H);
  memcpy(hp + a->wo.bih, b_ih, sizeof(float) * 3 * H);
  memcpy(hp + a->wo.bhh, b_hh, sizeof(float) * 3 * H);
  memcpy(hp + a->wo.b2, b2, sizeof(float) * A);
  if (tcb && (tc_supported(n, D, A, H, a->cfg.precision) || tcp_supported(n, D, A, H, a->cfg.precision) ||
              tcw_supported(n, D, A, H, a->cfg.precision)))
    tc_pack_weights(n, D, A, H, W1, b1, W_ih, b_ih, W_hh, b_hh, W2, b2, hp + a->wo.total);
}

static int upload_weights(marl_actor* a, const uint8_t* src, int image, cudaStream_t stream) {
  const marl_actor_config_t& c = a->cfg;
  const size_t tcb = tc_wpack_bytes(c.n_agents, c.obs_dim, c.n_actions, c.hidden);
  CU_TRY(cudaMemcpyAsync(a->state + a->so.wff[image], src, a->wo.total, cudaMemcpyHostToDevice, stream));
  if (tcb) CU_TRY(cudaMemcpyAsync(a->state + a->so.wpack[image], src + a->wo.total, tcb, cudaMemcpyHostToDevice, stream));
  return MARL_OK;
}

int marl_actor_set_weights(marl_actor_t* a, const float* W1, const float* b1, const float* W_ih,
                           const float* b_ih, const float* W_hh, const float* b_hh, const float* W2,
                           const float* b2, uint64_t version) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  if (!W1 || !b1 || !W_ih || !b_ih || !W_hh || !b_hh || !W2 || !b2) return fail(MARL_EINVAL, "a weight pointer is NULL");
  // The previous upload may still be in flight from this staging buffer, and enqueued steps may still read the image.
  CU_TRY(cudaStreamSynchronize(a->stream));
  if (a->pending) {  // a publication that has not taken effect is dropped
    CU_TRY(cudaStreamSynchronize(a->copy_stream));
    a->pending = false;
  }
  a->host_pack.resize(a->wo.total + tc_wpack_bytes(a->cfg.n_agents, a->cfg.obs_dim, a->cfg.n_actions, a->cfg.hidden));
  pack_weights_host(a, W1, b1, W_ih, b_ih, W_hh, b_hh, W2, b2, a->host_pack.data());
  const int rc = upload_weights(a, a->host_pack.data(), a->wslot, a->stream);
  if (rc) return rc;
  CU_TRY(cudaStreamSynchronize(a->stream));
  a->weights_version = version;
  a->have_weights = true;
  a->n_types = 1;  // one shared network again: the kernels chosen at creation
  a->agent_type_bits = 0;
  a->use_tc = a->tc_allowed;
  a->use_tcp = a->tcp_allowed;
  a->use_tc2 = a->tc2_allowed;
  return MARL_OK;
}

int marl_actor_set_weights_typed(marl_actor_t* a, int32_t n_types, const int32_t* agent_type, const float* W1,
                                 const float* b1, const float* W_ih, const float* b_ih, const float* W_hh,
                                 const float* b_hh, const float* W2, const float* b2, uint64_t version) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  if (!agent_type || !W1 || !b1 || !W_ih || !b_ih || !W_hh || !b_hh || !W2 || !b2) return fail(MARL_EINVAL, "a pointer is NULL");
  const marl_actor_config_t& c = a->cfg;
  const int cap = c.n_agent_types > 1 ? c.n_agent_types : 1;
  if (n_types < 1 || n_types > cap)
    return fail(MARL_EINVAL, "n_types=%d, but the actor was created for at most %d (n_agent_types)", n_types, cap);
  uint64_t bits = 0;
  for (int i = 0; i < c.n_agents; ++i) {
    if (agent_type[i] < 0 || agent_type[i] >= n_types)
      return fail(MARL_EINVAL, "agent_type[%d]=%d is outside [0, %d)", i, agent_type[i], n_types);
    bits |= (uint64_t)agent_type[i] << (2 * i);
  }
  CU_TRY(cudaStreamSynchronize(a->stream));
  if (a->pending) {
    CU_TRY(cudaStreamSynchronize(a->copy_stream));
    a->pending = false;
  }
  const int n = c.n_agents, D = c.obs_dim, A = c.n_actions, H = c.hidden, I = D + n + A;
  const size_t tcb = tc_wpack_bytes(n, D, A, H);
  a->host_pack.assign((size_t)n_types * a->wo.total + a->wo.total + tcb, 0);
  std::vector<uint8_t> one(a->wo.total + tcb);
  for (int k = 0; k < n_types; ++k) {  // the CUDA-core image of every type, one after the other
    pack_weights_host(a, W1 + (size_t)k * H * I, b1 + (size_t)k * H, W_ih + (size_t)k * 3 * H * H, b_ih + (size_t)k * 3 * H,
                      W_hh + (size_t)k * 3 * H * H, b_hh + (size_t)k * 3 * H, W2 + (size_t)k * A * H, b2 + (size_t)k * A,
                      one.data());
    memcpy(a->host_pack.data() + (size_t)k * a->wo.total, one.data(), a->wo.total);
  }
  CU_TRY(cudaMemcpyAsync(a->state + a->so.wff[a->wslot], a->host_pack.data(), (size_t)n_types * a->wo.total,
                         cudaMemcpyHostToDevice, a->stream));
  CU_TRY(cudaStreamSynchronize(a->stream));
  a->weights_version = version;
  a->have_weights = true;
  a->n_types = n_types;
  a->agent_type_bits = bits;
  a->use_tc = a->use_tcp = a->use_tc2 = false;  // per-type networks run on the CUDA-core kernel
  if (n_types == 1) {              // a single type is the shared network: its tensor-core image as well
    const int rc = upload_weights(a, one.data(), a->wslot, a->stream);
    if (rc) return rc;
    CU_TRY(cudaStreamSynchronize(a->stream));
    a->use_tc = a->tc_allowed;
    a->use_tcp = a->tcp_allowed;
    a->use_tc2 = a->tc2_allowed;
  }
  return MARL_OK;
}

int marl_actor_publish_weights(marl_actor_t* a, const float* W1, const float* b1, const float* W_ih,
                               const float* b_ih, const float* W_hh, const float* b_hh, const float* W2,
                               const float* b2, uint64_t version, uint64_t effective_step) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  if (!W1 || !b1 || !W_ih || !b_ih || !W_hh || !b_hh || !W2 || !b2) return fail(MARL_EINVAL, "a weight pointer is NULL");
  if (!a->have_weights) return fail(MARL_EINVAL, "marl_actor_set_weights has not been called");
  if (a->n_types > 1) return fail(MARL_EINVAL, "per-type networks are loaded: publish is for the shared network only");
  if (effective_step < a->step) return fail(MARL_EINVAL, "effective_step %llu is already enqueued (next step is %llu)",
                                            (unsigned long long)effective_step, (unsigned long long)a->step);
  if (!a->copy_stream) {
    CU_TRY(cudaStreamCreateWithFlags(&a->copy_stream, cudaStreamNonBlocking));
    CU_TRY(cudaEventCreateWithFlags(&a->upload_done, cudaEventDisableTiming));
    CU_TRY(cudaEventCreateWithFlags(&a->image_free, cudaEventDisableTiming));
    CU_TRY(cudaMallocHost(&a->host_pack2, a->wo.total + tc_wpack_bytes(a->cfg.n_agents, a->cfg.obs_dim, a->cfg.n_actions, a->cfg.hidden)));
  }
  // an earlier publication's copy reads host_pack2 and writes the same image: let it finish (it is replaced)
  CU_TRY(cudaStreamSynchronize(a->copy_stream));
  pack_weights_host(a, W1, b1, W_ih, b_ih, W_hh, b_hh, W2, b2, a->host_pack2);
  // the idle image was last read by steps enqueued before the previous switch
  if (a->image_free_recorded) CU_TRY(cudaStreamWaitEvent(a->copy_stream, a->image_free, 0));
  const int rc = upload_weights(a, a->host_pack2, a->wslot ^ 1, a->copy_stream);
  if (rc) return rc;
  CU_TRY(cudaEventRecord(a->upload_done, a->copy_stream));
  a->pending = true;
  a->pending_version = version;
  a->pending_step = effective_step;
  return MARL_OK;
}

uint64_t marl_actor_weights_version(const marl_actor_t* a) { return a ? a->weights_version : 0; }

static void fill_params(marl_actor* a, ActorParams& p) {
  const marl_actor_config_t& c = a->cfg;
  memset(&p, 0, sizeof(p));
  p.E = c.n_envs; p.n = c.n_agents; p.D = c.obs_dim; p.A = c.n_actions; p.H = c.hidden;
  p.I = c.obs_dim + c.n_agents + c.n_actions;
  p.L = c.ring_steps;
  p.S = c.ring_episodes / c.n_envs;
  p.prec = c.precision;
  p.seed = c.seed;
  uint8_t* st = a->state;
  const uint8_t* w = st + a->so.wff[a->wslot];
  p.W1T = reinterpret_cast<const float*>(w + a->wo.W1T);
  p.b1 = reinterpret_cast<const float*>(w + a->wo.b1);
  p.WihT = reinterpret_cast<const float*>(w + a->wo.WihT);
  p.bih = reinterpret_cast<const float*>(w + a->wo.bih);
  p.WhhT = reinterpret_cast<const float*>(w + a->wo.WhhT);
  p.bhh = reinterpret_cast<const float*>(w + a->wo.bhh);
  p.W2 = reinterpret_cast<const float*>(w + a->wo.W2);
  p.b2 = reinterpret_cast<const float*>(w + a->wo.b2);
  p.wpack = st + a->so.wpack[a->wslot];
  p.h = reinterpret_cast<float*>(st + a->so.h);
  p.last_action = reinterpret_cast<int32_t*>(st + a->so.last_action);
  p.slot = reinterpret_cast<int32_t*>(st + a->so.slot);
  p.pos = reinterpret_cast<int32_t*>(st + a->so.pos);
  p.ep_count = reinterpret_cast<long long*>(st + a->so.ep_count);
  p.ring = a->ring + a->ro.records;
  p.rl = a->rl;
  p.slot_stride = (long long)c.ring_steps * a->rl.rec_bytes;
  p.slot_epid = reinterpret_cast<long long*>(a->ring + a->ro.epid);
  p.slot_len = reinterpret_cast<int32_t*>(a->ring + a->ro.len);
  p.slot_complete = a->ring + a->ro.complete;
  p.counters = reinterpret_cast<unsigned long long*>(st + a->so.counters);
  p.status = reinterpret_cast<uint32_t*>(st + a->so.status);
  p.env_ids = nullptr;
  p.M = c.n_envs;
  p.lagged = 0;
  p.n_types = a->n_types;
  p.type_stride = (uint32_t)(a->wo.total / sizeof(float));
  p.agent_type_bits = a->agent_type_bits;
  p.trace_actions = a->trace_actions;
  p.trace_q = a->trace_q;
  p.trace_first = a->trace_next;
  p.trace_cap = (a->trace_actions || a->trace_q) ? a->trace_cap : 0;
}

// The published network becomes the one in use: the stream waits for its upload; the image used so far is idle once
// the work enqueued before this point is done.
static int switch_to_published(marl_actor* a) {
  CU_TRY(cudaStreamWaitEvent(a->stream, a->upload_done, 0));
  CU_TRY(cudaEventRecord(a->image_free, a->stream));
  a->image_free_recorded = true;
  a->wslot ^= 1;
  a->weights_version = a->pending_version;
  a->pending = false;
  return MARL_OK;
}

// Enqueues T steps reading inputs laid out [step][E]...; shared by every stepping entry point.
static int enqueue_steps(marl_actor* a, const float* obs, const uint8_t* avail, const float* reward,
                         const uint8_t* done, int T, bool eps_const, float eps, double eps_start,
                         double eps_end, int anneal, int32_t* actions_out) {
  if (!a->have_weights) return fail(MARL_EINVAL, "marl_actor_set_weights has not been called");
  if (a->step + (uint64_t)T > 0xFFFFFFFFull) return fail(MARL_EINVAL, "step counter would exceed 32 bits");
  const marl_actor_config_t& c = a->cfg;
  if (a->pending && a->step + (uint64_t)T > a->pending_step) {
    // A published network takes effect inside this span: the steps before it run on the current image, then the
    // stream waits for the upload (which has been running beside the earlier steps) and the images are swapped.
    const int T1 = a->pending_step > a->step ? (int)(a->pending_step - a->step) : 0;
    if (T1 > 0) {
      const int rc1 = enqueue_steps(a, obs, avail, reward, done, T1, eps_const, eps, eps_start, eps_end, anneal, nullptr);
      if (rc1) return rc1;
      obs += (size_t)T1 * c.n_envs * c.n_agents * c.obs_dim;
      avail += (size_t)T1 * c.n_envs * c.n_agents * c.n_actions;
      reward += (size_t)T1 * c.n_envs;
      done += (size_t)T1 * c.n_envs;
      T -= T1;
    }
    const int rcs = switch_to_published(a);
    if (rcs) return rcs;
  }
  ActorParams p;
  fill_params(a, p);
  p.T = T;
  p.t0 = (uint32_t)a->step;
  p.eps_const_mode = eps_const ? 1 : 0;
  p.eps_const = eps;
  p.eps_start = eps_start;
  p.eps_end = eps_end;
  p.anneal_steps = anneal;
  p.obs = obs; p.avail = avail; p.reward = reward; p.done = done;
  p.obs_step_stride = (long long)c.n_envs * c.n_agents * c.obs_dim;
  p.avail_step_stride = (long long)c.n_envs * c.n_agents * c.n_actions;
  p.env_step_stride = c.n_envs;
  p.actions_out = actions_out;
  int rc = 0;
  if (a->use_tcp || a->use_tc) {
    tc_tiling(c.n_envs, c.n_agents, a->sms, &p.ept, &p.num_tiles);
    if (a->use_tc2) rc = launch_actor_tc2(p, a->sms, a->stream);  // 0: not a launch for two resident tiles
    if (rc == 0 && a->use_tcp)  // 0: these pointers cannot be bulk-copied
      rc = c.hidden == 128 ? launch_actor_tcw(p, a->sms, a->stream) : launch_actor_tcp(p, a->sms, a->stream);
    // (the one-tile kernel bulk-copies the observations too; it copes with unaligned availability bytes itself)
    if (rc == 0 && a->use_tc && reinterpret_cast<uintptr_t>(obs) % 16 == 0) rc = launch_actor_tc(p, a->sms, a->stream);
  }
  if (rc == 0) {
    ffma_tiling(c.n_envs, c.n_agents, a->sms, &p.ept, &p.num_tiles);
    rc = launch_actor_ffma(p, a->sms, a->stream);
  }
  if (rc < 0) return fail(MARL_ECUDA, "actor kernel launch: %s", cudaGetErrorString((cudaError_t)(-rc)));
  a->launches += (uint64_t)rc;
  a->step += (uint64_t)T;
  if (a->trace_actions || a->trace_q) {
    const long long nx = (long long)a->trace_next + T;
    a->trace_next = nx > a->trace_cap ? a->trace_cap : (int32_t)nx;
  }
  return MARL_OK;
}

int marl_actor_step(marl_actor_t* a, const float* obs, const uint8_t* avail, const float* reward,
                    const uint8_t* done, float eps, int32_t* actions_out) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  if (!obs || !avail || !reward || !done) return fail(MARL_EINVAL, "an input pointer is NULL");
  if (!(eps >= 0.0f && eps <= 1.0f)) return fail(MARL_EINVAL, "eps must be in [0, 1]");
  return enqueue_steps(a, obs, avail, reward, done, 1, true, eps, 0, 0, 0, actions_out);
}

}  // extern "C"

// One step over a host list of environments; lagged: reward/done belong to each environment's previous action.
static int step_list(marl_actor* a, const int32_t* env_ids, int32_t M, const float* obs, const uint8_t* avail,
                     const float* reward, const uint8_t* done, float eps, int32_t* actions_out, bool lagged) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  if (!env_ids || !obs || !avail || !reward || !done) return fail(MARL_EINVAL, "an input pointer is NULL");
  if (!(eps >= 0.0f && eps <= 1.0f)) return fail(MARL_EINVAL, "eps must be in [0, 1]");
  const marl_actor_config_t& c = a->cfg;
  if (M < 1 || M > c.n_envs) return fail(MARL_EINVAL, "M=%d must be in [1, n_envs=%d]", M, c.n_envs);
  if (!a->have_weights) return fail(MARL_EINVAL, "marl_actor_set_weights has not been called");
  if (a->step + 1 > 0xFFFFFFFFull) return fail(MARL_EINVAL, "step counter would exceed 32 bits");
  // every listed environment exists and is listed once: two rows of one environment would race on its state
  a->id_seen.assign((size_t)c.n_envs, 0);
  for (int32_t x = 0; x < M; ++x) {
    const int32_t e = env_ids[x];
    if (e < 0 || e >= c.n_envs) return fail(MARL_EINVAL, "env_ids[%d]=%d is outside [0, %d)", x, e, c.n_envs);
    if (a->id_seen[e]) return fail(MARL_EINVAL, "env_ids[%d]=%d is listed twice", x, e);
    a->id_seen[e] = 1;
  }
  if (a->pending && a->step >= a->pending_step) {  // a published network is due
    const int rcs = switch_to_published(a);
    if (rcs) return rcs;
  }
  int32_t* d_ids = reinterpret_cast<int32_t*>(a->state + a->so.ids);
  // The caller's array (pageable or pinned) is free again when this call returns: the validated list is copied into
  // pinned staging owned by the actor and uploaded from there.  Two staging buffers take turns, each guarded by the
  // event of its last upload, so filling one never overwrites a copy that is still in flight.
  if (!a->ids_host[0]) {
    for (int i = 0; i < 2; ++i) {
      CU_TRY(cudaMallocHost(reinterpret_cast<void**>(&a->ids_host[i]), sizeof(int32_t) * (size_t)c.n_envs));
      CU_TRY(cudaEventCreateWithFlags(&a->ids_copied[i], cudaEventDisableTiming));
    }
  }
  const int ib = a->ids_next;
  a->ids_next ^= 1;
  if (a->ids_in_flight[ib]) CU_TRY(cudaEventSynchronize(a->ids_copied[ib]));
  memcpy(a->ids_host[ib], env_ids, sizeof(int32_t) * (size_t)M);
  CU_TRY(cudaMemcpyAsync(d_ids, a->ids_host[ib], sizeof(int32_t) * (size_t)M, cudaMemcpyHostToDevice, a->stream));
  CU_TRY(cudaEventRecord(a->ids_copied[ib], a->stream));
  a->ids_in_flight[ib] = true;
  ActorParams p;
  fill_params(a, p);
  p.T = 1;
  p.t0 = (uint32_t)a->step;
  p.eps_const_mode = 1;
  p.eps_const = eps;
  p.eps_start = p.eps_end = 0;
  p.anneal_steps = 0;
  p.obs = obs; p.avail = avail; p.reward = reward; p.done = done;
  p.obs_step_stride = p.avail_step_stride = p.env_step_stride = 0;
  p.actions_out = actions_out;
  p.env_ids = d_ids;
  p.M = M;
  p.lagged = lagged ? 1 : 0;
  int rc = 0;
  if (a->use_tcp) {  // 0: these pointers or this list length cannot be bulk-copied
    tc_tiling(M, c.n_agents, a->sms, &p.ept, &p.num_tiles);
    rc = c.hidden == 128 ? 0 : launch_actor_tcp(p, a->sms, a->stream);  // (the hidden-128 kernel takes dense launches only)
  }
  if (rc == 0) {
    ffma_tiling(M, c.n_agents, a->sms, &p.ept, &p.num_tiles);
    rc = launch_actor_ffma(p, a->sms, a->stream);
  }
  if (rc < 0) return fail(MARL_ECUDA, "actor kernel launch: %s", cudaGetErrorString((cudaError_t)(-rc)));
  a->launches += (uint64_t)rc;
  a->step += 1;
  if (a->trace_actions || a->trace_q) a->trace_next = a->trace_next + 1 > a->trace_cap ? a->trace_cap : a->trace_next + 1;
  return MARL_OK;
}

extern "C" {

int marl_actor_step_subset(marl_actor_t* a, const int32_t* env_ids, int32_t M, const float* obs,
                           const uint8_t* avail, const float* reward, const uint8_t* done, float eps,
                           int32_t* actions_out) {
  return step_list(a, env_ids, M, obs, avail, reward, done, eps, actions_out, false);
}

int marl_actor_step_lagged(marl_actor_t* a, const int32_t* env_ids, int32_t M, const float* obs,
                           const uint8_t* avail, const float* prev_reward, const uint8_t* prev_done, float eps,
                           int32_t* actions_out) {
  return step_list(a, env_ids, M, obs, avail, prev_reward, prev_done, eps, actions_out, true);
}

int marl_actor_step_host(marl_actor_t* a, const float* obs, const uint8_t* avail, const float* reward,
                         const uint8_t* done, float eps, int32_t* actions_out) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  if (!obs || !avail || !reward || !done) return fail(MARL_EINVAL, "an input pointer is NULL");
  if (!(eps >= 0.0f && eps <= 1.0f)) return fail(MARL_EINVAL, "eps must be in [0, 1]");
  const marl_actor_config_t& c = a->cfg;
  const WorkOffsets wo = work_offsets(c, 1);
  const size_t rows = (size_t)c.n_envs * c.n_agents;
  float* d_obs = reinterpret_cast<float*>(a->work + wo.obs);
  uint8_t* d_avail = a->work + wo.avail;
  float* d_reward = reinterpret_cast<float*>(a->work + wo.reward);
  uint8_t* d_done = a->work + wo.done;
  int32_t* d_act = reinterpret_cast<int32_t*>(a->work + wo.actions);
  CU_TRY(cudaMemcpyAsync(d_obs, obs, sizeof(float) * rows * c.obs_dim, cudaMemcpyHostToDevice, a->stream));
  CU_TRY(cudaMemcpyAsync(d_avail, avail, rows * c.n_actions, cudaMemcpyHostToDevice, a->stream));
  CU_TRY(cudaMemcpyAsync(d_reward, reward, sizeof(float) * c.n_envs, cudaMemcpyHostToDevice, a->stream));
  CU_TRY(cudaMemcpyAsync(d_done, done, (size_t)c.n_envs, cudaMemcpyHostToDevice, a->stream));
  const int rc = enqueue_steps(a, d_obs, d_avail, d_reward, d_done, 1, true, eps, 0, 0, 0, d_act);
  if (rc) return rc;
  if (actions_out)
    CU_TRY(cudaMemcpyAsync(actions_out, d_act, sizeof(int32_t) * rows, cudaMemcpyDeviceToHost, a->stream));
  CU_TRY(cudaStreamSynchronize(a->stream));
  return MARL_OK;
}

int marl_env_generate(const marl_actor_t* a_, const marl_synth_env_t* env, uint32_t t0, int32_t n_steps,
                      float* obs, uint8_t* avail, float* reward, uint8_t* done) {
  marl_actor* a = const_cast<marl_actor*>(a_);
  if (!a || !env) return fail(MARL_EINVAL, "actor or env is NULL");
  if (n_steps < 1) return fail(MARL_EINVAL, "n_steps must be >= 1");
  if (!obs || !avail || !reward || !done) return fail(MARL_EINVAL, "an output pointer is NULL");
  if ((reinterpret_cast<uintptr_t>(obs) | reinterpret_cast<uintptr_t>(avail) | reinterpret_cast<uintptr_t>(reward) |
       reinterpret_cast<uintptr_t>(done)) % 16)
    return fail(MARL_EALIGN, "environment arrays must be 16-byte aligned");
  if (env->obs_law != 0 && env->obs_law != 1) return fail(MARL_EINVAL, "obs_law must be 0 or 1");
  if (env->obs_law == 1 && 2 * a->cfg.obs_dim + 1 >= 65536) return fail(MARL_EINVAL, "obs_dim too large for law 1");
  const marl_actor_config_t& c = a->cfg;
  const int rc = launch_env_generate(*env, c.n_envs, c.n_agents, c.obs_dim, c.n_actions, t0, n_steps, obs, avail,
                                     reward, done, a->sms, a->stream);
  if (rc < 0) return fail(MARL_ECUDA, "environment kernel launch: %s", cudaGetErrorString((cudaError_t)(-rc)));
  a->launches += (uint64_t)rc;
  return MARL_OK;
}

int marl_rollout_staged(marl_actor_t* a, const float* obs, const uint8_t* avail, const float* reward,
                        const uint8_t* done, int32_t T, double eps_start, double eps_end, int32_t anneal_steps) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  if (!obs || !avail || !reward || !done) return fail(MARL_EINVAL, "an input pointer is NULL");
  if (T < 1) return fail(MARL_EINVAL, "T must be >= 1");
  if (!(eps_start >= 0.0 && eps_start <= 1.0 && eps_end >= 0.0 && eps_end <= 1.0))
    return fail(MARL_EINVAL, "eps must be in [0, 1]");
  return enqueue_steps(a, obs, avail, reward, done, T, false, 0.f, eps_start, eps_end, anneal_steps, nullptr);
}

int marl_rollout(marl_actor_t* a, const marl_synth_env_t* env, int32_t T, double eps_start, double eps_end,
                 int32_t anneal_steps) {
  if (!a || !env) return fail(MARL_EINVAL, "actor or env is NULL");
  if (T < 1) return fail(MARL_EINVAL, "T must be >= 1");
  const marl_actor_config_t& c = a->cfg;
  // Largest window of steps whose staging fits the work buffer.
  size_t W = 1;
  while (W < (size_t)T && work_offsets(c, W + 1).total <= a->work_bytes) {
    size_t W2 = W * 2 < (size_t)T ? W * 2 : (size_t)T;
    if (work_offsets(c, W2).total <= a->work_bytes) W = W2; else W += 1;
  }
  const WorkOffsets wo = work_offsets(c, W);
  float* d_obs = reinterpret_cast<float*>(a->work + wo.obs);
  uint8_t* d_avail = a->work + wo.avail;
  float* d_reward = reinterpret_cast<float*>(a->work + wo.reward);
  uint8_t* d_done = a->work + wo.done;
  int32_t left = T;
  while (left > 0) {
    const int32_t w = left < (int32_t)W ? left : (int32_t)W;
    int rc = marl_env_generate(a, env, (uint32_t)a->step, w, d_obs, d_avail, d_reward, d_done);
    if (rc) return rc;
    rc = marl_rollout_staged(a, d_obs, d_avail, d_reward, d_done, w, eps_start, eps_end, anneal_steps);
    if (rc) return rc;
    left -= w;
  }
  return MARL_OK;
}

int marl_actor_set_trace(marl_actor_t* a, int32_t* actions, float* q, int32_t capacity_steps) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  if (capacity_steps < 0) return fail(MARL_EINVAL, "capacity_steps must be >= 0");
  a->trace_actions = capacity_steps ? actions : nullptr;
  a->trace_q = capacity_steps ? q : nullptr;
  a->trace_cap = capacity_steps;
  a->trace_next = 0;
  return MARL_OK;
}

int marl_ring_view(const marl_actor_t* a, marl_ring_view_t* out) {
  if (!a || !out) return fail(MARL_EINVAL, "actor or out is NULL");
  const marl_actor_config_t& c = a->cfg;
  out->base = a->ring + a->ro.records;
  out->step_stride = a->rl.rec_bytes;
  out->slot_stride = (size_t)c.ring_steps * a->rl.rec_bytes;
  out->off_obs = a->rl.off_obs;
  out->off_avail = a->rl.off_avail;
  out->off_action = a->rl.off_action;
  out->off_q = a->rl.off_q;
  out->off_reward = a->rl.off_reward;
  out->off_done = a->rl.off_done;
  out->episodes = c.ring_episodes;
  out->steps = c.ring_steps;
  out->slots_per_env = c.ring_episodes / c.n_envs;
  out->n_envs = c.n_envs;
  out->n_agents = c.n_agents;
  out->obs_dim = c.obs_dim;
  out->n_actions = c.n_actions;
  out->reserved = 0;
  out->slot_epid = reinterpret_cast<int64_t*>(a->ring + a->ro.epid);
  out->slot_len = reinterpret_cast<int32_t*>(a->ring + a->ro.len);
  out->slot_complete = a->ring + a->ro.complete;
  return MARL_OK;
}

int marl_ring_sample(marl_actor_t* a, uint32_t draw_index, int32_t B, const marl_sample_batch_t* out) {
  if (!a || !out) return fail(MARL_EINVAL, "actor or out is NULL");
  if (B < 1 || B > 65535) return fail(MARL_EINVAL, "B must be in 1 .. 65535");
  const void* ptrs[9] = {out->obs, out->avail, out->action, out->q, out->reward, out->done, out->slot, out->len, out->epid};
  for (const void* q : ptrs) {
    if (!q) return fail(MARL_EINVAL, "a field of the batch is NULL");
    if (reinterpret_cast<uintptr_t>(q) % 16) return fail(MARL_EALIGN, "the fields of the batch must be 16-byte aligned");
  }
  const marl_actor_config_t& c = a->cfg;
  marl::SampleParams p;
  memset(&p, 0, sizeof(p));
  p.B = B; p.C = c.ring_episodes; p.L = c.ring_steps; p.n = c.n_agents; p.D = c.obs_dim; p.A = c.n_actions; p.E = c.n_envs;
  p.seed = c.seed;
  p.draw_index = draw_index;
  p.ring = a->ring + a->ro.records;
  p.rl = a->rl;
  p.slot_stride = (long long)c.ring_steps * a->rl.rec_bytes;
  p.slot_epid = reinterpret_cast<const long long*>(a->ring + a->ro.epid);
  p.slot_len = reinterpret_cast<const int32_t*>(a->ring + a->ro.len);
  p.slot_complete = a->ring + a->ro.complete;
  p.out = *out;
  const int rc = marl::launch_ring_sample(p, a->stream);
  if (rc < 0) return fail(MARL_ECUDA, "sampler kernel launch: %s", cudaGetErrorString((cudaError_t)(-rc)));
  a->launches += (uint64_t)rc;
  return MARL_OK;
}

int marl_actor_get_state(const marl_actor_t* a, marl_state_view_t* out) {
  if (!a || !out) return fail(MARL_EINVAL, "actor or out is NULL");
  uint8_t* st = a->state;
  out->h = reinterpret_cast<float*>(st + a->so.h);
  out->last_action = reinterpret_cast<int32_t*>(st + a->so.last_action);
  out->slot = reinterpret_cast<int32_t*>(st + a->so.slot);
  out->pos = reinterpret_cast<int32_t*>(st + a->so.pos);
  out->ep_count = reinterpret_cast<int64_t*>(st + a->so.ep_count);
  out->step = a->step;
  return MARL_OK;
}

int marl_actor_set_state(marl_actor_t* a, const marl_state_view_t* in) {
  if (!a || !in) return fail(MARL_EINVAL, "actor or in is NULL");
  if (!in->h || !in->last_action || !in->slot || !in->pos || !in->ep_count) return fail(MARL_EINVAL, "a state pointer is NULL");
  if (in->step > 0xFFFFFFFFull) return fail(MARL_EINVAL, "step counter exceeds 32 bits");
  const marl_actor_config_t& c = a->cfg;
  const size_t rows = (size_t)c.n_envs * c.n_agents;
  uint8_t* st = a->state;
  CU_TRY(cudaMemcpyAsync(st + a->so.h, in->h, sizeof(float) * rows * c.hidden, cudaMemcpyDeviceToDevice, a->stream));
  CU_TRY(cudaMemcpyAsync(st + a->so.last_action, in->last_action, sizeof(int32_t) * rows, cudaMemcpyDeviceToDevice, a->stream));
  CU_TRY(cudaMemcpyAsync(st + a->so.slot, in->slot, sizeof(int32_t) * c.n_envs, cudaMemcpyDeviceToDevice, a->stream));
  CU_TRY(cudaMemcpyAsync(st + a->so.pos, in->pos, sizeof(int32_t) * c.n_envs, cudaMemcpyDeviceToDevice, a->stream));
  CU_TRY(cudaMemcpyAsync(st + a->so.ep_count, in->ep_count, sizeof(int64_t) * c.n_envs, cudaMemcpyDeviceToDevice, a->stream));
  a->step = in->step;
  return MARL_OK;
}

int marl_actor_status(marl_actor_t* a, uint32_t* device_status, marl_counters_t* counters) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  uint64_t cnt[CNT_N];
  uint32_t st[4] = {0, 0, 0, 0};
  CU_TRY(cudaMemcpyAsync(cnt, a->state + a->so.counters, sizeof(cnt), cudaMemcpyDeviceToHost, a->stream));
  CU_TRY(cudaMemcpyAsync(st, a->state + a->so.status, sizeof(st), cudaMemcpyDeviceToHost, a->stream));
  CU_TRY(cudaStreamSynchronize(a->stream));
  if (device_status) *device_status = st[0] | (st[1] << 8);  // bits 8..: timeout diagnosis (barrier, warp)
  if (counters) {
    counters->agent_steps = cnt[CNT_AGENT_STEPS];
    counters->episodes = cnt[CNT_EPISODES];
    counters->explored = cnt[CNT_EXPLORED];
    counters->no_avail = cnt[CNT_NO_AVAIL];
    counters->truncated = cnt[CNT_TRUNCATED];
  }
  return MARL_OK;
}

int marl_actor_reset(marl_actor_t* a) {
  if (!a) return fail(MARL_EINVAL, "actor is NULL");
  return enqueue_reset(a);
}

const char* marl_actor_kernel_name(const marl_actor_t* a) { 
  if (!a) return "ffma";
  if (a->use_tc2) return "tcgen05-dual";
  if (a->use_tcp) return a->cfg.hidden == 128 ? "tcgen05-streamed" : "tcgen05-pipelined";
  return a->use_tc ? "tcgen05" : "ffma";
}

uint64_t marl_actor_launch_count(const marl_actor_t* a) { return a ? a->launches : 0; }

}  // extern "C"
