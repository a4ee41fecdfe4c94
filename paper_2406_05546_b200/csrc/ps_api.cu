// Host state machine and C ABI of the parameter-server hot path (see include/ps.h).
//
// The paper's coordination layer (ZooKeeper znodes for failure detection and for the references
// to weights and gradients, an object store holding the data) collapses, inside one process on
// one GPU, into host integers and device buffers: a weight version counter, a ring of retained
// weight versions for stale readers, a linear gradient queue whose slots the grad step writes in
// place, pinned host checkpoint slots, and replica weight buffers for the server chain.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "kernels.h"
#include "ps.h"

static_assert(PS_PARAM_COUNT == psk::P && PS_PARAM_STRIDE == psk::P_PAD, "layout constants");
static_assert(PS_MAX_WORKERS == psk::MAX_WORKERS && PS_MAX_RING == psk::MAX_RING, "limits");

namespace {

constexpr int MAX_SPLIT = 16;
constexpr uint64_t ALIGN = 256;
constexpr uint64_t VEC_BYTES = (uint64_t)psk::P_PAD * sizeof(float);

thread_local std::string g_err;

struct QueueMeta { int32_t worker; uint64_t base_version; uint64_t step; };
struct Replica { float* buf; uint64_t version; bool alive; };

uint64_t align_up(uint64_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }

// Carves consecutive aligned blocks out of a base address (or just measures when base == 0).
struct Carver {
  uint64_t base, off = 0;
  explicit Carver(void* p) : base((uint64_t)p) {}
  template <typename T> T* take(uint64_t bytes) {
    off = align_up(off);
    T* p = reinterpret_cast<T*>(base + off);
    off += bytes;
    return p;
  }
};

}  // namespace

struct ps_ctx {
  ps_config cfg;
  cudaStream_t st;
  float* ring[psk::MAX_RING];
  std::vector<Replica> replicas;
  float* partial;
  float* queue;
  float* coef_dev;                      // [queue_slots] per-gradient factors of a treated apply
  float* norm_part;                     // [queue_slots][NORM_CHUNKS] partial sums of squares
  cudaEvent_t coef_uploaded = nullptr;  // the staged factors have left coef_host
  psk::Workspace ws;
  float* x_stage[2]; int32_t* y_stage[2]; float* loss_stage[2]; int32_t* argmax_stage[2];   // two sets: two ticks may be in flight
  uint32_t* status_dev;
  // pinned
  std::vector<float*> ckpt_buf;
  std::vector<uint64_t> ckpt_version;   // parallel to ckpt_buf
  std::vector<int> ckpt_order;          // slot indices, oldest first
  float* io_stage;
  float* coef_host;                     // per-gradient factors of a treated apply, staged for upload
  uint32_t* status_host;
  // state
  uint64_t version = 0, oldest = 0;
  bool up = true, weights_lost = false;
  int64_t queue_len = 0, reserved = 0, applied_total = 0, launches = 0;
  int32_t w_tick = 0;
  std::vector<QueueMeta> meta;
  uint32_t drop_thresh = 0;
  psk::Profiler prof;
  psk::SideStreams side;
  // rounded copies of the dense-layer weights: which snapshots they were made from, and in which state of the weights
  uint64_t weights_epoch = 1, prep_epoch = 0;
  const float* prep_theta[psk::MAX_GROUPS] = {nullptr};
  int prep_n = 0;
  // ps_tick_host copies its inputs in on a stream of its own, chunk by chunk, while earlier chunks compute
  cudaStream_t copy_st = nullptr;
  cudaEvent_t copy_ev[8] = {nullptr};          // [set][chunk]
  cudaEvent_t stage_free[2] = {nullptr, nullptr}, tick_done[2] = {nullptr, nullptr};
  struct { bool used = false; ps_apply_result res = {0, 0, 0, 0}; } inflight[2];
  uint64_t ticks_submitted = 0, ticks_waited = 0;
  double prof_ms[psk::K_COUNT] = {0};
  int64_t prof_n[psk::K_COUNT] = {0};
};

namespace {

int32_t fail(int32_t code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}

int32_t cuda_fail(cudaError_t e, const char* what) {
  return fail(PS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define CUDA_TRY(expr)                                   \
  do {                                                   \
    cudaError_t e_ = (expr);                             \
    if (e_ != cudaSuccess) return cuda_fail(e_, #expr);  \
  } while (0)

int32_t check_cfg(const ps_config* c) {
  if (!c) return fail(PS_ERR_BAD_ARG, "config is NULL");
  if (c->max_workers < 1 || c->max_workers > PS_MAX_WORKERS) return fail(PS_ERR_BAD_ARG, "max_workers must be 1..%d", PS_MAX_WORKERS);
  if (c->max_batch < 1 || c->max_batch > 4096) return fail(PS_ERR_BAD_ARG, "max_batch must be 1..4096");
  if (c->ring_depth < 1 || c->ring_depth > PS_MAX_RING) return fail(PS_ERR_BAD_ARG, "ring_depth must be 1..%d", PS_MAX_RING);
  if (c->ckpt_every < 0 || c->ckpt_slots < 0 || (c->ckpt_every > 0 && c->ckpt_slots < 1)) return fail(PS_ERR_BAD_ARG, "checkpoint settings");
  if (c->chain_len < 1 || c->chain_len > 8) return fail(PS_ERR_BAD_ARG, "chain_len must be 1..8");
  if (c->replicate_every < 1) return fail(PS_ERR_BAD_ARG, "replicate_every must be >= 1");
  if (c->external_store != 0 && c->external_store != 1) return fail(PS_ERR_BAD_ARG, "external_store must be 0 or 1");
  if (c->precision != PS_FP32 && c->precision != PS_BF16) return fail(PS_ERR_BAD_ARG, "precision %d is not built (PS_FP32 and PS_BF16 are)", c->precision);
  if (!(c->dropout_p >= 0.f) || !(c->dropout_p < 1.f)) return fail(PS_ERR_BAD_ARG, "dropout_p must be in [0,1)");
  if (c->queue_slots < 1) return fail(PS_ERR_BAD_ARG, "queue_slots must be >= 1");
  return PS_OK;
}

// Lays the context's device and pinned buffers out over the two caller-owned blocks.
void layout(ps_ctx* x, const ps_config& c, void* arena, void* pinned, uint64_t* arena_bytes, uint64_t* pinned_bytes) {
  const uint64_t rows = (uint64_t)c.max_workers * c.max_batch;
  // partial-sum slots per worker: one per block of CONV_SPB samples, or four per range of the tensor-core
  // filter-gradient kernel (at most (b - 1) / 16 + 2 ranges meet a worker)
  const uint64_t chunks = ((uint64_t)c.max_batch + psk::CONV_SPB - 1) / psk::CONV_SPB + 8;
  Carver a(arena);
  for (int i = 0; i < c.ring_depth; ++i) { float* p = a.take<float>(VEC_BYTES); if (x) x->ring[i] = p; }
  for (int i = 0; i + 1 < c.chain_len; ++i) { float* p = a.take<float>(VEC_BYTES); if (x) x->replicas.push_back({p, 0, true}); }
  float* partial = a.take<float>(VEC_BYTES * MAX_SPLIT);
  float* queue = a.take<float>(VEC_BYTES * (uint64_t)c.queue_slots);
  float* coef_dev = a.take<float>((uint64_t)c.queue_slots * 4);
  float* norm_part = a.take<float>((uint64_t)c.queue_slots * psk::NORM_CHUNKS * 4);
  psk::Workspace ws;
  const uint64_t p1_elems = c.precision != PS_FP32 ? psk::P1_PLANE_ELEMS : psk::P1_ELEMS;
  ws.p1 = a.take<float>(rows * p1_elems * 4);
  ws.code1 = a.take<uint8_t>(rows * psk::P1_ELEMS);
  ws.p2 = a.take<float>(rows * psk::FLAT * 4);
  ws.code2 = a.take<uint8_t>(rows * psk::FLAT);
  ws.d = a.take<float>(rows * psk::HID * 4);
  ws.da1 = a.take<float>(rows * psk::HID * 4);
  ws.dz = a.take<float>(rows * psk::DZ_STRIDE * 4);
  ws.dp2 = a.take<float>(rows * psk::FLAT * 4);
  ws.dp1 = a.take<float>(rows * psk::P1_ELEMS * 4);
  ws.part2 = a.take<float>((uint64_t)c.max_workers * chunks * psk::C2_GRAD * 4);
  ws.part1 = a.take<float>((uint64_t)c.max_workers * 8 * chunks * psk::C1_GRAD * 4);
  ws.partf = a.take<float>((uint64_t)c.max_workers * psk::FC2_SPLIT * psk::FC_PART * 4);
  ws.status = a.take<uint32_t>(ALIGN);
  ws.w1r = ws.w1tr = nullptr;
  if (c.precision != PS_FP32) {
    const uint64_t groups = std::min<uint64_t>(psk::MAX_GROUPS, std::min<uint64_t>(c.max_workers, c.ring_depth));
    ws.w1r = a.take<float>(groups * psk::HID * psk::FLAT * 4);
    ws.w1tr = a.take<float>(groups * psk::HID * psk::FLAT * 4);
  }
  float* x_stage[2]; int32_t* y_stage[2]; float* loss_stage[2]; int32_t* argmax_stage[2];
  for (int k = 0; k < 2; ++k) {
    x_stage[k] = a.take<float>(rows * PS_IMAGE_PIXELS * 4);
    y_stage[k] = a.take<int32_t>(rows * 4);
    loss_stage[k] = a.take<float>((uint64_t)c.max_workers * 4);
    argmax_stage[k] = a.take<int32_t>(rows * 4);
  }
  Carver h(pinned);
  for (int i = 0; i < c.ckpt_slots; ++i) { float* p = h.take<float>(VEC_BYTES); if (x) x->ckpt_buf.push_back(p); }
  float* io_stage = h.take<float>(VEC_BYTES);
  float* coef_host = h.take<float>((uint64_t)c.queue_slots * 4);
  uint32_t* status_host = h.take<uint32_t>(ALIGN);
  if (x) {
    x->partial = partial; x->queue = queue; x->ws = ws; x->status_dev = ws.status;
    x->coef_dev = coef_dev; x->norm_part = norm_part; x->coef_host = coef_host;
    for (int k = 0; k < 2; ++k) { x->x_stage[k] = x_stage[k]; x->y_stage[k] = y_stage[k]; x->loss_stage[k] = loss_stage[k]; x->argmax_stage[k] = argmax_stage[k]; }
    x->io_stage = io_stage; x->status_host = status_host;
  }
  if (arena_bytes) *arena_bytes = align_up(a.off);
  if (pinned_bytes) *pinned_bytes = align_up(h.off);
}

float* head(ps_ctx* x) { return x->ring[x->version % (uint64_t)x->cfg.ring_depth]; }

void advance_oldest(ps_ctx* x) {
  uint64_t depth = (uint64_t)x->cfg.ring_depth;
  if (x->version + 1 > depth && x->oldest < x->version + 1 - depth) x->oldest = x->version + 1 - depth;
}

Replica* first_live(ps_ctx* x) {
  for (auto& r : x->replicas) if (r.alive) return &r;
  return nullptr;
}

int32_t do_checkpoint(ps_ctx* x) {
  if (x->ckpt_buf.empty()) return fail(PS_ERR_BAD_ARG, "no checkpoint slots configured");
  int slot;
  if (x->ckpt_order.size() < x->ckpt_buf.size()) {
    slot = (int)x->ckpt_order.size();
  } else {
    slot = x->ckpt_order.front();
    x->ckpt_order.erase(x->ckpt_order.begin());
  }
  CUDA_TRY(cudaMemcpyAsync(x->ckpt_buf[slot], head(x), VEC_BYTES, cudaMemcpyDeviceToHost, x->st));
  x->ckpt_version[slot] = x->version;
  x->ckpt_order.push_back(slot);
  return PS_OK;
}

// Chain replication with relaxed consistency (paper, design section on chain-replicated servers): at a replication
// event the frontend hands its weights to the next live server and waits for that server only; the hop to the server
// behind it completes with the following event.  After `events` events the i-th live server behind the frontend
// (i = 0 first) therefore holds the version replicated i events before the latest one.  This routine does the part
// that moves existing contents down the chain, on the stream and BEFORE the kernel (or copy) that writes the
// newest versions: server i takes what server i - events held.  Servers i < events are written by the caller, which
// sets their versions with set_replica_versions().
int32_t shift_chain(ps_ctx* x, int events) {
  std::vector<Replica*> live;
  for (auto& r : x->replicas) if (r.alive) live.push_back(&r);
  for (int i = (int)live.size() - 1; i >= events; --i) {
    CUDA_TRY(cudaMemcpyAsync(live[i]->buf, live[i - events]->buf, VEC_BYTES, cudaMemcpyDeviceToDevice, x->st));
    live[i]->version = live[i - events]->version;
  }
  return PS_OK;
}

// The live servers behind the frontend, nearest first.
std::vector<Replica*> live_chain(ps_ctx* x) {
  std::vector<Replica*> live;
  for (auto& r : x->replicas) if (r.alive) live.push_back(&r);
  return live;
}

}  // namespace

extern "C" {

const char* ps_last_error(ps_ctx*) { return g_err.c_str(); }

int32_t ps_query_bytes(const ps_config* cfg, uint64_t* arena_bytes, uint64_t* pinned_bytes) {
  int32_t rc = check_cfg(cfg);
  if (rc != PS_OK) return rc;
  layout(nullptr, *cfg, nullptr, nullptr, arena_bytes, pinned_bytes);
  return PS_OK;
}

int32_t ps_create(const ps_config* cfg, const float* init_params_host, ps_ctx** out) {
  int32_t rc = check_cfg(cfg);
  if (rc != PS_OK) return rc;
  if (!init_params_host || !out) return fail(PS_ERR_BAD_ARG, "NULL argument");
  if (!cfg->arena || ((uint64_t)cfg->arena % ALIGN) != 0) return fail(PS_ERR_BAD_ARG, "arena must be a 256-byte aligned device pointer");
  if (!cfg->pinned) return fail(PS_ERR_BAD_ARG, "pinned block is NULL");
  uint64_t need_a = 0, need_p = 0;
  layout(nullptr, *cfg, nullptr, nullptr, &need_a, &need_p);
  if (cfg->arena_bytes < need_a) return fail(PS_ERR_ARENA_TOO_SMALL, "arena has %llu bytes, %llu needed", (unsigned long long)cfg->arena_bytes, (unsigned long long)need_a);
  if (cfg->pinned_bytes < need_p) return fail(PS_ERR_ARENA_TOO_SMALL, "pinned block has %llu bytes, %llu needed", (unsigned long long)cfg->pinned_bytes, (unsigned long long)need_p);
  ps_ctx* x = new (std::nothrow) ps_ctx();
  if (!x) return fail(PS_ERR_BAD_ARG, "out of host memory");
  x->cfg = *cfg;
  x->st = (cudaStream_t)cfg->stream;
  layout(x, *cfg, cfg->arena, cfg->pinned, nullptr, nullptr);
  x->ckpt_version.assign(x->ckpt_buf.size(), 0);
  double t = std::floor((double)cfg->dropout_p * 4294967296.0);
  x->drop_thresh = t <= 0.0 ? 0u : (t >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)t);
  if (psk::configure_grad_kernels() != 0 || psk::configure_tc5_kernels() != 0 || psk::configure_conv5_kernels() != 0 || psk::configure_conv1_kernels() != 0 || psk::configure_dw5_kernels() != 0 || psk::configure_c1d5_kernels() != 0) { delete x; return fail(PS_ERR_CUDA, "kernel configuration failed: %s", cudaGetErrorString(cudaGetLastError())); }
  if (cfg->precision != PS_FP32) {
    // two side streams let independent branches of the backward pass overlap (they allocate no device memory)
    bool ok = cudaStreamCreateWithFlags(&x->side.s1, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&x->side.s2, cudaStreamNonBlocking) == cudaSuccess;
    cudaEvent_t* evs[4] = {&x->side.fork1, &x->side.join1, &x->side.fork2, &x->side.join2};
    for (auto ev : evs) ok = ok && cudaEventCreateWithFlags(ev, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { delete x; return fail(PS_ERR_CUDA, "side stream set-up failed: %s", cudaGetErrorString(cudaGetLastError())); }
  }
  {
    bool ok = cudaStreamCreateWithFlags(&x->copy_st, cudaStreamNonBlocking) == cudaSuccess;
    for (auto& ev : x->copy_ev) ok = ok && cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess;
    for (auto& ev : x->stage_free) ok = ok && cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess;
    for (auto& ev : x->tick_done) ok = ok && cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&x->coef_uploaded, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { delete x; return fail(PS_ERR_CUDA, "copy stream set-up failed: %s", cudaGetErrorString(cudaGetLastError())); }
  }
  std::memcpy(x->io_stage, init_params_host, sizeof(float) * PS_PARAM_COUNT);
  std::memset(x->io_stage + PS_PARAM_COUNT, 0, sizeof(float) * (PS_PARAM_STRIDE - PS_PARAM_COUNT));
  cudaError_t e = cudaMemcpyAsync(x->ring[0], x->io_stage, VEC_BYTES, cudaMemcpyHostToDevice, x->st);
  for (auto& r : x->replicas)
    if (e == cudaSuccess) e = cudaMemcpyAsync(r.buf, x->io_stage, VEC_BYTES, cudaMemcpyHostToDevice, x->st);
  if (e == cudaSuccess) e = cudaMemsetAsync(x->status_dev, 0, ALIGN, x->st);
  // tensor-core path: the zero borders of the plane-layout activations are written once, here
  if (e == cudaSuccess && cfg->precision != PS_FP32)
    e = cudaMemsetAsync(x->ws.p1, 0, (uint64_t)cfg->max_workers * cfg->max_batch * psk::P1_PLANE_ELEMS * 4, x->st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(x->st);
  if (e != cudaSuccess) { delete x; return cuda_fail(e, "ps_create upload"); }
  *out = x;
  return PS_OK;
}

int32_t ps_destroy(ps_ctx* x) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  cudaError_t e = cudaStreamSynchronize(x->st);
  if (x->side.s1) { cudaStreamSynchronize(x->side.s1); cudaStreamDestroy(x->side.s1); }
  if (x->side.s2) { cudaStreamSynchronize(x->side.s2); cudaStreamDestroy(x->side.s2); }
  for (cudaEvent_t ev : {x->side.fork1, x->side.join1, x->side.fork2, x->side.join2}) if (ev) cudaEventDestroy(ev);
  if (x->copy_st) { cudaStreamSynchronize(x->copy_st); cudaStreamDestroy(x->copy_st); }
  for (cudaEvent_t ev : x->copy_ev) if (ev) cudaEventDestroy(ev);
  for (cudaEvent_t ev : x->stage_free) if (ev) cudaEventDestroy(ev);
  for (cudaEvent_t ev : x->tick_done) if (ev) cudaEventDestroy(ev);
  if (x->coef_uploaded) cudaEventDestroy(x->coef_uploaded);
  delete x;
  if (e != cudaSuccess) return cuda_fail(e, "ps_destroy");
  return PS_OK;
}

int32_t ps_pull_snapshot(ps_ctx* x, int32_t worker, int32_t lag, ps_snapshot* out) {
  if (!x || !out) return fail(PS_ERR_BAD_ARG, "NULL argument");
  if (worker < 0 || lag < 0) return fail(PS_ERR_BAD_ARG, "negative worker or lag");
  if (x->weights_lost || (!x->up && !x->cfg.external_store)) return fail(PS_ERR_DOWN, "server is down and its weights died with it");
  if ((uint64_t)lag > x->version || x->version - (uint64_t)lag < x->oldest)
    return fail(PS_ERR_VERSION_EVICTED, "version head-%d is not retained (head %llu, oldest %llu)", lag, (unsigned long long)x->version, (unsigned long long)x->oldest);
  uint64_t v = x->version - (uint64_t)lag;
  out->version = v;
  out->dev_ptr = x->ring[v % (uint64_t)x->cfg.ring_depth];
  return PS_OK;
}

int32_t ps_queue_reserve(ps_ctx* x, int32_t n, int64_t* slot_ids) {
  if (!x || !slot_ids || n < 1) return fail(PS_ERR_BAD_ARG, "bad argument");
  if (!x->up && !x->cfg.external_store) return fail(PS_ERR_DOWN, "server is down");
  if (x->queue_len + n > x->cfg.queue_slots) return fail(PS_ERR_QUEUE_FULL, "queue holds %lld of %lld, %d more requested", (long long)x->queue_len, (long long)x->cfg.queue_slots, n);
  x->reserved = n;
  for (int i = 0; i < n; ++i) slot_ids[i] = x->queue_len + i;
  return PS_OK;
}

int32_t ps_slot_ptr(ps_ctx* x, int64_t slot_id, float** out) {
  if (!x || !out || slot_id < 0 || slot_id >= x->cfg.queue_slots) return fail(PS_ERR_BAD_ARG, "bad slot");
  *out = x->queue + slot_id * (int64_t)psk::P_PAD;
  return PS_OK;
}

// Sorts the workers of a call by weight snapshot (workers sharing a pointer become one group) and fills the tables
// the kernels take.  grad destinations: queue slots, rows of grads_dev, or none (evaluation).
static int32_t build_tables(ps_ctx* x, int32_t W, const ps_snapshot* snaps, const int32_t* worker_ids, const int64_t* slot_ids,
                            float* grads_dev, psk::WorkerTable& wt, psk::GroupTable& gt) {
  int group_of[PS_MAX_WORKERS];
  gt.n_groups = 0;
  for (int w = 0; w < W; ++w) {
    if (!snaps[w].dev_ptr) return fail(PS_ERR_BAD_ARG, "snapshot %d has no weights", w);
    int g = 0;
    while (g < gt.n_groups && gt.theta[g] != snaps[w].dev_ptr) ++g;
    if (g == gt.n_groups) {
      if (g == psk::MAX_GROUPS) return fail(PS_ERR_BAD_ARG, "more than %d distinct snapshots", psk::MAX_GROUPS);
      gt.theta[gt.n_groups++] = snaps[w].dev_ptr;
    }
    group_of[w] = g;
  }
  int s = 0;
  for (int g = 0; g < gt.n_groups; ++g) {
    gt.first[g] = s;
    for (int w = 0; w < W; ++w) {
      if (group_of[w] != g) continue;
      if (slot_ids) {
        int64_t id = slot_ids[w];
        if (id < x->queue_len || id >= x->queue_len + x->reserved) return fail(PS_ERR_BAD_ARG, "slot %lld is not reserved", (long long)id);
        wt.grad[s] = x->queue + id * (int64_t)psk::P_PAD;
      } else {
        wt.grad[s] = grads_dev ? grads_dev + (int64_t)w * psk::P_PAD : nullptr;
      }
      wt.wid[s] = worker_ids ? worker_ids[w] : w;
      wt.src[s] = w;
      wt.group[s] = (int16_t)g;
      ++s;
    }
  }
  gt.first[gt.n_groups] = W;
  if (x->cfg.precision != PS_FP32 && gt.n_groups > std::min(x->cfg.max_workers, x->cfg.ring_depth))
    return fail(PS_ERR_BAD_ARG, "%d distinct snapshots but the tensor-core workspace holds ring_depth = %d", gt.n_groups, x->cfg.ring_depth);
  return PS_OK;
}

// The rounded / transposed copies of the dense-layer weights are reused while the same snapshots hold the same weights.
static int prep_is_current(ps_ctx* x, const psk::GroupTable& gt) {
  bool same = x->prep_epoch == x->weights_epoch && x->prep_n == gt.n_groups;
  for (int g = 0; g < gt.n_groups && same; ++g) same = x->prep_theta[g] == gt.theta[g];
  return same ? 1 : 0;
}
static void prep_done(ps_ctx* x, const psk::GroupTable& gt) {
  x->prep_epoch = x->weights_epoch; x->prep_n = gt.n_groups;
  for (int g = 0; g < gt.n_groups; ++g) x->prep_theta[g] = gt.theta[g];
}

int32_t workers_grad_step(ps_ctx* x, int32_t W, int32_t b, const ps_snapshot* snaps, const int32_t* worker_ids,
                          const float* x_dev, const int32_t* y_dev, uint64_t seed, uint64_t step,
                          const int64_t* slot_ids, float* grads_dev, float* loss_dev, int32_t* argmax_dev) {
  if (!x || !snaps || !worker_ids || !x_dev || !y_dev || !loss_dev || !argmax_dev) return fail(PS_ERR_BAD_ARG, "NULL argument");
  if (W < 1 || W > x->cfg.max_workers || b < 1 || b > x->cfg.max_batch) return fail(PS_ERR_BAD_ARG, "W=%d, b=%d outside 1..%d, 1..%d", W, b, x->cfg.max_workers, x->cfg.max_batch);
  if (!slot_ids && !grads_dev) return fail(PS_ERR_BAD_ARG, "neither slot_ids nor grads_dev given");
  psk::GroupTable gt;
  psk::WorkerTable wt;
  int32_t rc = build_tables(x, W, snaps, worker_ids, slot_ids, grads_dev, wt, gt);
  if (rc != PS_OK) return rc;
  psk::GradStepArgs a;
  a.W = W; a.b = b; a.x = x_dev; a.y = y_dev; a.loss = loss_dev; a.argmax = argmax_dev;
  a.seed = seed; a.step = step; a.drop_p = x->cfg.dropout_p; a.drop_thresh = x->drop_thresh;
  a.precision = x->cfg.precision;
  if (a.precision != PS_FP32 && ((uintptr_t)x_dev & 15) != 0) return fail(PS_ERR_BAD_ARG, "x_dev must be 16-byte aligned on the tensor-core path");
  a.skip_prep_w1 = prep_is_current(x, gt);
  int n = psk::launch_grad_step(a, wt, gt, x->ws, x->st, x->prof.on ? psk::SideStreams() : x->side, &x->prof);
  if (n >= 0 && a.precision != PS_FP32) prep_done(x, gt);
  if (n < 0) return cuda_fail(cudaGetLastError(), "grad step launch");
  x->launches += n;
  return PS_OK;
}

int32_t workers_grad_step_summed(ps_ctx* x, int32_t W, int32_t b, const ps_snapshot* snaps, const int32_t* worker_ids,
                                 const float* x_dev, const int32_t* y_dev, uint64_t seed, uint64_t step, float* grad_sum_dev,
                                 float* loss_dev, int32_t* argmax_dev) {
  if (!x || !snaps || !worker_ids || !x_dev || !y_dev || !grad_sum_dev || !loss_dev || !argmax_dev) return fail(PS_ERR_BAD_ARG, "NULL argument");
  if (W < 1 || W > x->cfg.max_workers || b < 1 || b > x->cfg.max_batch) return fail(PS_ERR_BAD_ARG, "W=%d, b=%d outside 1..%d, 1..%d", W, b, x->cfg.max_workers, x->cfg.max_batch);
  if (((uintptr_t)grad_sum_dev & 15) != 0) return fail(PS_ERR_BAD_ARG, "grad_sum_dev must be 16-byte aligned");
  psk::GroupTable gt;
  psk::WorkerTable wt;
  int32_t rc = build_tables(x, W, snaps, worker_ids, nullptr, nullptr, wt, gt);
  if (rc != PS_OK) return rc;
  if (gt.n_groups != 1) return fail(PS_ERR_BAD_ARG, "the summed step needs every worker on the same snapshot (%d distinct ones given)", gt.n_groups);
  psk::GradStepArgs a;
  a.W = W; a.b = b; a.x = x_dev; a.y = y_dev; a.loss = loss_dev; a.argmax = argmax_dev;
  a.seed = seed; a.step = step; a.drop_p = x->cfg.dropout_p; a.drop_thresh = x->drop_thresh;
  a.precision = x->cfg.precision;
  if (a.precision != PS_FP32 && ((uintptr_t)x_dev & 15) != 0) return fail(PS_ERR_BAD_ARG, "x_dev must be 16-byte aligned on the tensor-core path");
  a.skip_prep_w1 = prep_is_current(x, gt);
  psk::SummedStep sum;
  sum.grad_sum = grad_sum_dev;
  sum.super_part = x->partial;          // the reduction scratch is free between applies
  sum.n_super = 1;
  for (int g = MAX_SPLIT; g >= 1; --g)
    if (W % g == 0) { sum.n_super = g; break; }
  int n = psk::launch_grad_step(a, wt, gt, x->ws, x->st, x->prof.on ? psk::SideStreams() : x->side, &x->prof, &sum);
  if (n >= 0 && a.precision != PS_FP32) prep_done(x, gt);
  if (n < 0) return cuda_fail(cudaGetLastError(), "summed grad step launch");
  x->launches += n;
  return PS_OK;
}

int32_t ps_apply_summed(ps_ctx* x, const float* grad_sum_dev, int32_t n_workers, float lr, float scale, ps_apply_result* out) {
  if (!x || !grad_sum_dev || n_workers < 1) return fail(PS_ERR_BAD_ARG, "bad argument");
  if (!x->up || x->weights_lost) return fail(PS_ERR_DOWN, "server is down");
  if (x->queue_len != 0) return fail(PS_ERR_BAD_ARG, "the queue holds %lld gradients: apply them first", (long long)x->queue_len);
  if (((uintptr_t)grad_sum_dev & 15) != 0) return fail(PS_ERR_BAD_ARG, "grad_sum_dev must be 16-byte aligned");
  const uint64_t depth = (uint64_t)x->cfg.ring_depth, R = (uint64_t)x->cfg.replicate_every;
  Replica* rep = first_live(x);
  ps_apply_result res = {0, x->version, 0, 0};
  psk::SumApplyArgs a;
  a.queue = grad_sum_dev; a.K = 1;
  a.theta_in = head(x);
  a.theta_out = x->ring[(x->version + 1) % depth];
  const bool mirror = rep && ((x->version + 1) % R == 0);
  if (mirror) { int32_t rc = shift_chain(x, 1); if (rc != PS_OK) return rc; }
  a.replica = mirror ? rep->buf : nullptr;
  a.coef = lr * scale / (float)n_workers;
  a.partial = x->partial; a.max_split = 1;
  a.coef_k = nullptr;
  int n = psk::launch_sum_apply(a, x->st, &x->prof);
  if (n < 0) return cuda_fail(cudaGetLastError(), "apply launch");
  x->launches += n;
  x->version += 1;
  x->weights_epoch++;
  advance_oldest(x);
  if (mirror) { rep->version = x->version; res.replicated = 1; }
  if (x->cfg.ckpt_every > 0 && x->version % (uint64_t)x->cfg.ckpt_every == 0) {
    int32_t rc = do_checkpoint(x); if (rc != PS_OK) return rc; res.checkpointed = 1;
  }
  x->applied_total += n_workers;
  res.applied = n_workers;
  res.new_version = x->version;
  if (out) *out = res;
  return PS_OK;
}

int32_t workers_eval(ps_ctx* x, int32_t W, int32_t b, const ps_snapshot* snaps, const float* x_dev, const int32_t* y_dev,
                     float* loss_dev, int32_t* argmax_dev, int32_t* correct_dev) {
  if (!x || !snaps || !x_dev || !y_dev || !loss_dev || !argmax_dev || !correct_dev) return fail(PS_ERR_BAD_ARG, "NULL argument");
  if (W < 1 || W > x->cfg.max_workers || b < 1 || b > x->cfg.max_batch) return fail(PS_ERR_BAD_ARG, "W=%d, b=%d outside 1..%d, 1..%d", W, b, x->cfg.max_workers, x->cfg.max_batch);
  psk::GroupTable gt;
  psk::WorkerTable wt;
  int32_t rc = build_tables(x, W, snaps, nullptr, nullptr, nullptr, wt, gt);
  if (rc != PS_OK) return rc;
  psk::GradStepArgs a;
  a.W = W; a.b = b; a.x = x_dev; a.y = y_dev; a.loss = loss_dev; a.argmax = argmax_dev;
  a.seed = 0; a.step = 0; a.drop_p = 0.f; a.drop_thresh = 0u;      // inference: nothing is dropped, nothing rescaled
  a.precision = x->cfg.precision;
  if (a.precision != PS_FP32 && ((uintptr_t)x_dev & 15) != 0) return fail(PS_ERR_BAD_ARG, "x_dev must be 16-byte aligned on the tensor-core path");
  a.skip_prep_w1 = prep_is_current(x, gt);
  int n = psk::launch_eval(a, wt, gt, x->ws, correct_dev, x->st, &x->prof);
  if (n >= 0 && a.precision != PS_FP32) prep_done(x, gt);
  if (n < 0) return cuda_fail(cudaGetLastError(), "evaluation launch");
  x->launches += n;
  return PS_OK;
}

int32_t ps_dropout_mask(ps_ctx* x, uint64_t seed, int32_t worker_id, uint64_t step, int32_t b, uint8_t* keep_dev) {
  if (!x || !keep_dev || b < 1 || b > 4096) return fail(PS_ERR_BAD_ARG, "bad argument");
  if (((uint64_t)keep_dev & 3) != 0) return fail(PS_ERR_BAD_ARG, "keep_dev must be 4-byte aligned");
  int n = psk::launch_dropout_mask(seed, (uint32_t)worker_id, step, b, x->drop_thresh, keep_dev, x->st, &x->prof);
  if (n < 0) return cuda_fail(cudaGetLastError(), "dropout mask launch");
  x->launches += n;
  return PS_OK;
}

int32_t ps_enqueue(ps_ctx* x, int32_t n, const int64_t* slot_ids, const float* grads_dev,
                   const int32_t* worker_ids, const uint64_t* base_versions, uint64_t step) {
  if (!x || n < 1 || !worker_ids || !base_versions) return fail(PS_ERR_BAD_ARG, "bad argument");
  if (!slot_ids && !grads_dev) return fail(PS_ERR_BAD_ARG, "neither slot_ids nor grads_dev given");
  if (!x->up && !x->cfg.external_store) return fail(PS_ERR_DOWN, "server is down");
  if (x->queue_len + n > x->cfg.queue_slots) return fail(PS_ERR_QUEUE_FULL, "queue holds %lld of %lld", (long long)x->queue_len, (long long)x->cfg.queue_slots);
  if (x->queue_len > 0 && n != x->w_tick) return fail(PS_ERR_BAD_ARG, "gradients per enqueue changed from %d to %d while the queue is not empty", x->w_tick, n);
  if (slot_ids) {
    if (n > x->reserved) return fail(PS_ERR_BAD_ARG, "%d slots given but %lld reserved", n, (long long)x->reserved);
    for (int i = 0; i < n; ++i)
      if (slot_ids[i] != x->queue_len + i) return fail(PS_ERR_BAD_ARG, "slot_ids must be the reserved slots in order");
  } else {
    int r = psk::launch_copy_rows(x->queue + x->queue_len * (int64_t)psk::P_PAD, grads_dev, n, x->st, &x->prof);
    if (r < 0) return cuda_fail(cudaGetLastError(), "enqueue copy");
    x->launches += r;
  }
  for (int i = 0; i < n; ++i) x->meta.push_back({worker_ids[i], base_versions[i], step});
  x->w_tick = n;
  x->queue_len += n;
  x->reserved = 0;
  return PS_OK;
}

int32_t ps_checkpoint(ps_ctx* x, uint64_t* version_out) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  if (!x->up || x->weights_lost) return fail(PS_ERR_DOWN, "server is down");
  int32_t rc = do_checkpoint(x);
  if (rc == PS_OK && version_out) *version_out = x->version;
  return rc;
}

int32_t ps_replicate(ps_ctx* x, uint64_t* version_out) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  if (!x->up || x->weights_lost) return fail(PS_ERR_DOWN, "server is down");
  Replica* r = first_live(x);
  if (!r) return fail(PS_ERR_NO_REPLICA, "no live replica");
  int32_t rc = shift_chain(x, 1);
  if (rc != PS_OK) return rc;
  CUDA_TRY(cudaMemcpyAsync(r->buf, head(x), VEC_BYTES, cudaMemcpyDeviceToDevice, x->st));
  r->version = x->version;
  if (version_out) *version_out = x->version;
  return PS_OK;
}

// One server step.  clip_norm > 0 and / or staleness_alpha > 0 switch the stale-gradient treatments on: every queued
// gradient then gets a factor of its own (learning rate included), staged on the host, uploaded, and, for clipping,
// multiplied on the device by min(1, clip_norm / ||g||) after one pass over the queue that takes the norms.
static int32_t apply_impl(ps_ctx* x, ps_mode mode, float lr, float scale, const int32_t* order, float clip_norm,
                          float staleness_alpha, ps_apply_result* out) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  if (!x->up || x->weights_lost) return fail(PS_ERR_DOWN, "server is down");
  if (mode != PS_SYNC && mode != PS_ASYNC && mode != PS_REPLAY) return fail(PS_ERR_BAD_ARG, "unknown mode %d", (int)mode);
  const int64_t K = x->queue_len;
  ps_apply_result res = {0, x->version, 0, 0};
  x->reserved = 0;
  if (K == 0) { if (out) *out = res; return PS_OK; }
  if (order) {
    std::vector<uint8_t> seen((size_t)K, 0);
    for (int64_t k = 0; k < K; ++k) {
      if (order[k] < 0 || order[k] >= K || seen[(size_t)order[k]]) return fail(PS_ERR_BAD_ARG, "order is not a permutation of the queue");
      seen[(size_t)order[k]] = 1;
    }
  }
  const bool treated = clip_norm > 0.f || staleness_alpha > 0.f;
  if (treated) {
    // factor of the gradient in queue slot k: the step size of its mode times 1 / (1 + alpha * staleness), where the
    // staleness is the version the update is applied to minus the version the worker had read
    const double step = mode == PS_ASYNC ? (double)lr * (double)scale
                                         : (double)lr * (double)scale / (double)(mode == PS_SYNC ? K : (int64_t)x->w_tick);
    CUDA_TRY(cudaEventSynchronize(x->coef_uploaded));      // an earlier treated apply has read the staging buffer
    for (int64_t j = 0; j < K; ++j) {
      const int64_t k = (mode == PS_ASYNC && order) ? order[j] : j;
      const uint64_t applied_to = x->version + (mode == PS_ASYNC ? (uint64_t)j : 0u);
      const uint64_t base = x->meta[(size_t)k].base_version;
      if (staleness_alpha > 0.f && base > applied_to)
        return fail(PS_ERR_BAD_ARG, "gradient %lld claims base version %llu, newer than the version %llu it is applied to",
                    (long long)k, (unsigned long long)base, (unsigned long long)applied_to);
      const double tau = staleness_alpha > 0.f ? (double)(applied_to - base) : 0.0;
      x->coef_host[k] = (float)(step / (1.0 + (double)staleness_alpha * tau));
    }
    CUDA_TRY(cudaMemcpyAsync(x->coef_dev, x->coef_host, (size_t)K * sizeof(float), cudaMemcpyHostToDevice, x->st));
    CUDA_TRY(cudaEventRecord(x->coef_uploaded, x->st));
    if (clip_norm > 0.f) {
      int n = psk::launch_clip_factors(x->queue, K, clip_norm, x->coef_dev, x->norm_part, x->st, &x->prof);
      if (n < 0) return cuda_fail(cudaGetLastError(), "clipping launch");
      x->launches += n;
    }
  }
  const uint64_t depth = (uint64_t)x->cfg.ring_depth;
  const uint64_t R = (uint64_t)x->cfg.replicate_every;
  Replica* rep = first_live(x);
  if (mode == PS_SYNC || mode == PS_REPLAY) {
    psk::SumApplyArgs a;
    a.queue = x->queue; a.K = K;
    a.theta_in = head(x);
    a.theta_out = x->ring[(x->version + 1) % depth];
    const bool mirror = rep && ((x->version + 1) % R == 0);
    if (mirror) { int32_t rc = shift_chain(x, 1); if (rc != PS_OK) return rc; }
    a.replica = mirror ? rep->buf : nullptr;
    a.coef = lr * scale / (float)(mode == PS_SYNC ? K : (int64_t)x->w_tick);
    a.partial = x->partial; a.max_split = MAX_SPLIT;
    a.coef_k = treated ? x->coef_dev : nullptr;
    int n = psk::launch_sum_apply(a, x->st, &x->prof);
    if (n < 0) return cuda_fail(cudaGetLastError(), "apply launch");
    x->launches += n;
    x->version += 1;
    x->weights_epoch++;
    advance_oldest(x);
    if (mirror) { rep->version = x->version; res.replicated = 1; }
    if (x->cfg.ckpt_every > 0 && x->version % (uint64_t)x->cfg.ckpt_every == 0) {
      int32_t rc = do_checkpoint(x); if (rc != PS_OK) return rc; res.checkpointed = 1;
    }
  } else {
    // Ordered application in segments that end at checkpoint boundaries, so that the version to
    // be checkpointed is the head when it is copied out.
    int64_t pos = 0;
    while (pos < K) {
      int64_t seg = std::min<int64_t>(psk::ASYNC_SEG, K - pos);
      if (x->cfg.ckpt_every > 0) {
        uint64_t ce = (uint64_t)x->cfg.ckpt_every;
        uint64_t to_ckpt = ce - x->version % ce;
        seg = std::min<int64_t>(seg, (int64_t)to_ckpt);
      }
      psk::AsyncApplyArgs a;
      psk::AsyncOrder ord;
      a.queue = x->queue; a.K = (int)seg; a.theta_in = head(x);
      for (int i = 0; i < psk::MAX_RING; ++i) a.ring[i] = i < x->cfg.ring_depth ? x->ring[i] : nullptr;
      a.ring_depth = x->cfg.ring_depth; a.v0 = x->version;
      a.first_stored = (int)std::max<int64_t>(0, seg - (int64_t)depth);
      a.n_mirror = 0; a.coef = lr * scale;
      a.coef_k = treated ? x->coef_dev : nullptr;
      if (rep) {
        // replication events inside this segment: versions that are multiples of R.  The i-th live server behind
        // the frontend receives the version of the i-th latest event if that version is produced here; what the
        // servers further down receive comes from the servers in front of them (shift_chain, before the launch).
        const uint64_t last = (x->version + (uint64_t)seg) / R * R;
        const int events = (int)((x->version + (uint64_t)seg) / R - x->version / R);
        if (events > 0) {
          int32_t rc = shift_chain(x, events); if (rc != PS_OK) return rc;
          std::vector<Replica*> live = live_chain(x);
          for (int i = 0; i < (int)live.size() && i < events; ++i) {
            const uint64_t v = last - (uint64_t)i * R;
            a.mirror_k[a.n_mirror] = (int)(v - x->version - 1);
            a.replica[a.n_mirror] = live[i]->buf;
            ++a.n_mirror;
            live[i]->version = v;
          }
          res.replicated += events;
        }
      }
      for (int64_t u = 0; u < seg; ++u) ord.slot[u] = order ? order[pos + u] : (int32_t)(pos + u);
      int n = psk::launch_async_apply(a, ord, x->st, &x->prof);
      if (n < 0) return cuda_fail(cudaGetLastError(), "async apply launch");
      x->launches += n;
      x->version += (uint64_t)seg;
      x->weights_epoch++;
      advance_oldest(x);
      if (x->cfg.ckpt_every > 0 && x->version % (uint64_t)x->cfg.ckpt_every == 0) {
        int32_t rc = do_checkpoint(x); if (rc != PS_OK) return rc; res.checkpointed += 1;
      }
      pos += seg;
    }
  }
  x->queue_len = 0;
  x->meta.clear();
  x->applied_total += K;
  res.applied = K;
  res.new_version = x->version;
  if (out) *out = res;
  return PS_OK;
}

int32_t ps_apply(ps_ctx* x, ps_mode mode, float lr, float scale, const int32_t* order, ps_apply_result* out) {
  return apply_impl(x, mode, lr, scale, order, 0.f, 0.f, out);
}

int32_t ps_apply_stale(ps_ctx* x, ps_mode mode, float lr, float scale, const int32_t* order, float clip_norm,
                       float staleness_alpha, ps_apply_result* out) {
  if (!(clip_norm >= 0.f) || !(staleness_alpha >= 0.f)) return fail(PS_ERR_BAD_ARG, "clip_norm and staleness_alpha must be >= 0");
  return apply_impl(x, mode, lr, scale, order, clip_norm, staleness_alpha, out);
}

int32_t ps_kill(ps_ctx* x, int32_t server) {
  if (!x || server < 0) return fail(PS_ERR_BAD_ARG, "bad argument");
  if (server == 0) {
    x->up = false;
    x->reserved = 0;
    if (!x->cfg.external_store) {
      x->weights_lost = true;
      x->queue_len = 0;
      x->meta.clear();
    }
    return PS_OK;
  }
  int live = 0;
  for (auto& r : x->replicas) {
    if (!r.alive) continue;
    if (++live == server) { r.alive = false; return PS_OK; }
  }
  return fail(PS_ERR_BAD_ARG, "no live server %d behind the frontend", server);
}

int32_t ps_restore(ps_ctx* x, uint64_t* version_out) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  if (x->cfg.external_store) {
    x->up = true;
    if (version_out) *version_out = x->version;
    return PS_OK;
  }
  if (x->ckpt_order.empty()) return fail(PS_ERR_NO_CHECKPOINT, "no checkpoint has been taken");
  int slot = x->ckpt_order.back();
  uint64_t v = x->ckpt_version[slot];
  CUDA_TRY(cudaMemcpyAsync(x->ring[v % (uint64_t)x->cfg.ring_depth], x->ckpt_buf[slot], VEC_BYTES, cudaMemcpyHostToDevice, x->st));
  x->version = v; x->oldest = v;
  x->weights_epoch++;
  x->queue_len = 0; x->reserved = 0; x->meta.clear();
  x->up = true; x->weights_lost = false;
  if (version_out) *version_out = v;
  return PS_OK;
}

int32_t ps_failover(ps_ctx* x, uint64_t* version_out) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  size_t i = 0;
  while (i < x->replicas.size() && !x->replicas[i].alive) ++i;
  if (i == x->replicas.size()) return fail(PS_ERR_NO_REPLICA, "no live replica");
  Replica r = x->replicas[i];
  // The new frontend's warm weights become the head: swap buffers, no bytes move.
  uint64_t slot = r.version % (uint64_t)x->cfg.ring_depth;
  x->ring[slot] = r.buf;   // the dead frontend's buffer in that slot is retired
  x->replicas.erase(x->replicas.begin(), x->replicas.begin() + (long)i + 1);
  x->version = r.version; x->oldest = r.version;
  x->weights_epoch++;
  x->queue_len = 0; x->reserved = 0; x->meta.clear();
  x->up = true; x->weights_lost = false;
  if (version_out) *version_out = r.version;
  return PS_OK;
}

int32_t ps_import_params(ps_ctx* x, const float* host_in) {
  if (x) x->weights_epoch++;
  if (!x || !host_in) return fail(PS_ERR_BAD_ARG, "NULL argument");
  if (x->weights_lost) return fail(PS_ERR_DOWN, "server is down");
  CUDA_TRY(cudaStreamSynchronize(x->st));
  std::memcpy(x->io_stage, host_in, sizeof(float) * PS_PARAM_COUNT);
  std::memset(x->io_stage + PS_PARAM_COUNT, 0, sizeof(float) * (PS_PARAM_STRIDE - PS_PARAM_COUNT));
  CUDA_TRY(cudaMemcpyAsync(head(x), x->io_stage, VEC_BYTES, cudaMemcpyHostToDevice, x->st));
  CUDA_TRY(cudaStreamSynchronize(x->st));
  return PS_OK;
}

int32_t ps_export_params(ps_ctx* x, int32_t which, float* host_out, uint64_t* version_out) {
  if (!x || !host_out) return fail(PS_ERR_BAD_ARG, "NULL argument");
  const float* src_dev = nullptr;
  const float* src_host = nullptr;
  uint64_t v = 0;
  if (which == 0) {
    if (x->weights_lost) return fail(PS_ERR_DOWN, "the frontend's weights are lost");
    src_dev = head(x); v = x->version;
  } else if (which < 0) {
    int want = -which, live = 0;
    for (auto& r : x->replicas)
      if (r.alive && ++live == want) { src_dev = r.buf; v = r.version; }
    if (!src_dev) return fail(PS_ERR_NO_REPLICA, "no live replica %d", want);
  } else if (which >= 1000) {
    int j = which - 1000;
    if (j >= (int)x->ckpt_order.size()) return fail(PS_ERR_NO_CHECKPOINT, "no checkpoint %d", j);
    int slot = x->ckpt_order[x->ckpt_order.size() - 1 - (size_t)j];
    src_host = x->ckpt_buf[slot]; v = x->ckpt_version[slot];
  } else {
    return fail(PS_ERR_BAD_ARG, "unknown selector %d", which);
  }
  if (src_dev) {
    CUDA_TRY(cudaMemcpyAsync(x->io_stage, src_dev, VEC_BYTES, cudaMemcpyDeviceToHost, x->st));
    src_host = x->io_stage;
  }
  CUDA_TRY(cudaStreamSynchronize(x->st));
  std::memcpy(host_out, src_host, sizeof(float) * PS_PARAM_COUNT);
  if (version_out) *version_out = v;
  return PS_OK;
}

int32_t ps_stats(ps_ctx* x, ps_stats_t* out) {
  if (!x || !out) return fail(PS_ERR_BAD_ARG, "NULL argument");
  CUDA_TRY(cudaMemcpyAsync(x->status_host, x->status_dev, sizeof(uint32_t), cudaMemcpyDeviceToHost, x->st));
  CUDA_TRY(cudaStreamSynchronize(x->st));
  out->version = x->version;
  out->oldest_version = x->oldest;
  out->queue_len = x->queue_len;
  out->applied_total = x->applied_total;
  out->up = x->up ? 1 : 0;
  int live = 0;
  for (auto& r : x->replicas) live += r.alive ? 1 : 0;
  out->live_replicas = live;
  out->checkpoints = (int32_t)x->ckpt_order.size();
  out->device_status = *x->status_host;
  Replica* r = first_live(x);
  out->replica_version = r ? r->version : 0;
  out->last_ckpt_version = x->ckpt_order.empty() ? 0 : x->ckpt_version[x->ckpt_order.back()];
  out->kernel_launches = x->launches;
  if (out->device_status != 0) return fail(PS_ERR_DEVICE_STATUS, "device status 0x%x (bit 0: label outside 0..9; bit 1: a bounded wait in a tensor-core kernel gave up)", out->device_status);
  return PS_OK;
}

int32_t ps_selftest_wait_timeout(ps_ctx* x, int64_t limit_cycles) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  if (limit_cycles < 1 || limit_cycles > 2000000000ll) return fail(PS_ERR_BAD_ARG, "limit_cycles must be 1..2e9");
  int n = psk::launch_wait_timeout_probe(x->status_dev, (long long)limit_cycles, x->st);
  if (n < 0) return cuda_fail(cudaGetLastError(), "probe launch");
  x->launches += n;
  return PS_OK;
}

int32_t ps_profile(ps_ctx* x, int32_t enable) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  CUDA_TRY(cudaStreamSynchronize(x->st));
  x->prof.collect(x->prof_ms, x->prof_n);
  x->prof.on = enable != 0;
  if (enable) for (int i = 0; i < psk::K_COUNT; ++i) { x->prof_ms[i] = 0; x->prof_n[i] = 0; }
  return PS_OK;
}

int32_t ps_profile_read(ps_ctx* x, int32_t kernel, const char** name, double* total_ms, int64_t* launches) {
  if (!x || kernel < 0) return fail(PS_ERR_BAD_ARG, "bad argument");
  if (kernel >= psk::K_COUNT) return fail(PS_ERR_BAD_ARG, "no kernel %d", kernel);
  CUDA_TRY(cudaStreamSynchronize(x->st));
  x->prof.collect(x->prof_ms, x->prof_n);
  if (name) *name = psk::kernel_name(kernel);
  if (total_ms) *total_ms = x->prof_ms[kernel];
  if (launches) *launches = x->prof_n[kernel];
  return PS_OK;
}

int32_t ps_tick_host_submit(ps_ctx* x, int32_t W, int32_t b, const int32_t* lags, const float* x_host, const int32_t* y_host,
                            uint64_t seed, uint64_t step, int32_t apply_mode, float lr, float scale, const int32_t* order,
                            float* loss_host, int32_t* argmax_host) {
  if (!x || !x_host || !y_host || !loss_host) return fail(PS_ERR_BAD_ARG, "NULL argument");
  if (W < 1 || W > x->cfg.max_workers || b < 1 || b > x->cfg.max_batch) return fail(PS_ERR_BAD_ARG, "W or b out of range");
  const int set = (int)(x->ticks_submitted & 1);
  if (x->inflight[set].used) return fail(PS_ERR_BAD_ARG, "two ticks are already in flight: call ps_tick_host_wait first");
  ps_snapshot snaps[PS_MAX_WORKERS];
  int32_t ids[PS_MAX_WORKERS];
  int64_t slots[PS_MAX_WORKERS];
  uint64_t bases[PS_MAX_WORKERS];
  for (int w = 0; w < W; ++w) {
    int32_t rc = ps_pull_snapshot(x, w, lags ? lags[w] : 0, &snaps[w]);
    if (rc != PS_OK) return rc;
    ids[w] = w;
    bases[w] = snaps[w].version;
  }
  int32_t rc = ps_queue_reserve(x, W, slots);
  if (rc != PS_OK) return rc;
  const size_t rows = (size_t)W * b;
  float* xs = x->x_stage[set];
  int32_t* ys = x->y_stage[set];
  // The inputs go in on the copy stream in up to four chunks of workers; the grad step of a chunk starts as soon as
  // its chunk has landed, so most of the host-to-device copy hides behind the computation of earlier chunks, and the
  // copies of this tick behind the previous tick's work.  This staging set was last read by the tick before the
  // previous one; the copy stream waits for that tick's grad step.
  if (x->ticks_submitted >= 2) CUDA_TRY(cudaStreamWaitEvent(x->copy_st, x->stage_free[set], 0));
  const int n_chunks = W >= 8 ? 4 : 1, per = (W + n_chunks - 1) / n_chunks;
  for (int c = 0; c < n_chunks; ++c) {
    const int w0 = c * per, w1 = std::min(W, w0 + per);
    if (w0 >= w1) break;
    const size_t r0 = (size_t)w0 * b, nr = (size_t)(w1 - w0) * b;
    CUDA_TRY(cudaMemcpyAsync(xs + r0 * PS_IMAGE_PIXELS, x_host + r0 * PS_IMAGE_PIXELS, nr * PS_IMAGE_PIXELS * sizeof(float), cudaMemcpyHostToDevice, x->copy_st));
    CUDA_TRY(cudaMemcpyAsync(ys + r0, y_host + r0, nr * sizeof(int32_t), cudaMemcpyHostToDevice, x->copy_st));
    CUDA_TRY(cudaEventRecord(x->copy_ev[4 * set + c], x->copy_st));
  }
  for (int c = 0; c < n_chunks; ++c) {
    const int w0 = c * per, w1 = std::min(W, w0 + per);
    if (w0 >= w1) break;
    const size_t r0 = (size_t)w0 * b;
    CUDA_TRY(cudaStreamWaitEvent(x->st, x->copy_ev[4 * set + c], 0));
    rc = workers_grad_step(x, w1 - w0, b, snaps + w0, ids + w0, xs + r0 * PS_IMAGE_PIXELS, ys + r0, seed, step,
                           slots + w0, nullptr, x->loss_stage[set] + w0, x->argmax_stage[set] + r0);
    if (rc != PS_OK) { cudaStreamSynchronize(x->copy_st); return rc; }
  }
  CUDA_TRY(cudaEventRecord(x->stage_free[set], x->st));
  rc = ps_enqueue(x, W, slots, nullptr, ids, bases, step);
  if (rc != PS_OK) return rc;
  ps_apply_result res = {0, x->version, 0, 0};
  if (apply_mode >= 0) {
    rc = ps_apply(x, (ps_mode)apply_mode, lr, scale, order, &res);
    if (rc != PS_OK) return rc;
  }
  CUDA_TRY(cudaMemcpyAsync(loss_host, x->loss_stage[set], (size_t)W * sizeof(float), cudaMemcpyDeviceToHost, x->st));
  if (argmax_host) CUDA_TRY(cudaMemcpyAsync(argmax_host, x->argmax_stage[set], rows * sizeof(int32_t), cudaMemcpyDeviceToHost, x->st));
  CUDA_TRY(cudaEventRecord(x->tick_done[set], x->st));
  x->inflight[set].used = true;
  x->inflight[set].res = res;
  x->ticks_submitted++;
  return PS_OK;
}

int32_t ps_tick_host_wait(ps_ctx* x, ps_apply_result* out) {
  if (!x) return fail(PS_ERR_BAD_ARG, "ctx is NULL");
  const int set = (int)(x->ticks_waited & 1);
  if (x->ticks_waited == x->ticks_submitted || !x->inflight[set].used) return fail(PS_ERR_BAD_ARG, "no tick is in flight");
  CUDA_TRY(cudaEventSynchronize(x->tick_done[set]));
  if (out) *out = x->inflight[set].res;
  x->inflight[set].used = false;
  x->ticks_waited++;
  return PS_OK;
}

int32_t ps_tick_host(ps_ctx* x, int32_t W, int32_t b, const int32_t* lags, const float* x_host, const int32_t* y_host,
                     uint64_t seed, uint64_t step, int32_t apply_mode, float lr, float scale, const int32_t* order,
                     float* loss_host, int32_t* argmax_host, ps_apply_result* out) {
  if (x && x->ticks_waited != x->ticks_submitted) return fail(PS_ERR_BAD_ARG, "a submitted tick is still in flight: call ps_tick_host_wait first");
  int32_t rc = ps_tick_host_submit(x, W, b, lags, x_host, y_host, seed, step, apply_mode, lr, scale, order, loss_host, argmax_host);
  if (rc != PS_OK) return rc;
  return ps_tick_host_wait(x, out);
}

}  // extern "C"
