// Internal launch interface between the host state machine and the sm_100a kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

namespace psk {

constexpr int P = 813258;
constexpr int P_PAD = 813312;          // floats per stored parameter / gradient vector
constexpr int P_VEC4 = P_PAD / 4;      // 203,328 float4 columns
constexpr int MAX_WORKERS = 256;
constexpr int MAX_RING = 16;
constexpr int MAX_GROUPS = 16;
constexpr int MAX_CHAIN = 8;           // servers in a replication chain, the frontend included

constexpr int OFF_C1W = 0, OFF_C1B = 144, OFF_C2W = 160, OFF_C2B = 4768;
constexpr int OFF_F1W = 4800, OFF_F1B = 807616, OFF_F2W = 808128, OFF_F2B = 813248;

constexpr int IMG = 28, C1 = 16, H1 = 14, C2 = 32, H2 = 7;
constexpr int P1_ELEMS = C1 * H1 * H1;   // 3136
constexpr int P1_PLANE_ELEMS = 2 * 256 * 4;   // 32-bit words of one sample's p1 in the tensor-core plane layout (8 KB of BF16)
constexpr int FLAT = C2 * H2 * H2;       // 1568
constexpr int HID = 512, NCLS = 10;
constexpr int DZ_STRIDE = 16;            // logits gradient row, padded
constexpr int CONV_SPB = 4;              // samples per block in the conv backward kernels
constexpr int C2_GRAD = 4608 + 32, C1_GRAD = 144 + 16;
constexpr int FC2_SPLIT = 1;             // blocks per worker in the output-layer kernel, each with its own partial sums (at 128 registers x 512 threads one block fills an SM, so more blocks only queue)
constexpr int FC_PART = NCLS * HID + HID + NCLS + 2;   // fc2.w, fc1.b, fc2.b gradients, loss sum, padding

constexpr uint32_t STATUS_BAD_LABEL = 1u;
constexpr uint32_t STATUS_WAIT_TIMEOUT = 2u;   // a bounded barrier wait in a tensor-core kernel gave up

// Optional per-kernel timing: when switched on, every launch is bracketed by two CUDA events on
// the launching stream; totals per kernel are read back after a synchronisation.
enum KernelId {
  K_CONV1_FWD = 0, K_CONV2_FWD, K_FC1_FWD, K_FC2_FWD_BWD, K_FC1_DW, K_FC1_DX, K_CONV2_BWD, K_CONV1_BWD,
  K_CONV_GRAD_REDUCE, K_SUM_APPLY_DIRECT, K_SUM_PARTIAL, K_SUM_FINISH, K_ASYNC_APPLY, K_COPY_ROWS,
  K_DROPOUT_MASK, K_CONV2_DW, K_PREP_W1, K_SQ_NORM, K_COEF_FINISH, K_EVAL_FINISH, K_COUNT
};
const char* kernel_name(int id);

struct Profiler {
  bool on = false;
  struct Rec { int id; cudaEvent_t a, b; };
  std::vector<Rec> recs;
  std::vector<cudaEvent_t> free_events;
  cudaEvent_t get() {
    if (!free_events.empty()) { cudaEvent_t e = free_events.back(); free_events.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
  }
  void begin(int id, cudaStream_t st) {
    if (!on) return;
    Rec r{id, get(), get()};
    cudaEventRecord(r.a, st);
    recs.push_back(r);
  }
  void end(cudaStream_t st) {
    if (!on) return;
    cudaEventRecord(recs.back().b, st);
  }
  // Caller has synchronised the stream.  Adds elapsed times into ms[K_COUNT] / n[K_COUNT] and recycles events.
  void collect(double* ms, int64_t* n) {
    for (auto& r : recs) {
      float t = 0.f;
      if (cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) { ms[r.id] += t; n[r.id] += 1; }
      free_events.push_back(r.a);
      free_events.push_back(r.b);
    }
    recs.clear();
  }
  ~Profiler() {
    for (auto& r : recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (auto e : free_events) cudaEventDestroy(e);
  }
};

// Per-call tables passed by value as kernel parameters.
// Workers are processed in "sorted" order: workers sharing a weight snapshot are adjacent, so
// that a group's samples form one contiguous block of activation rows.
struct WorkerTable {
  float* grad[MAX_WORKERS];     // destination gradient vector (P_PAD floats) of sorted worker s
  int32_t wid[MAX_WORKERS];     // logical worker id (dropout key)
  int32_t src[MAX_WORKERS];     // index of the worker in the caller's arrays (x, y, loss, argmax)
  int16_t group[MAX_WORKERS];   // group of sorted worker s
};

struct GroupTable {
  const float* theta[MAX_GROUPS];  // weight snapshot of the group
  int32_t first[MAX_GROUPS + 1];   // first sorted worker of the group; first[n_groups] = W
  int32_t n_groups;
};

// Activation workspace carved from the arena (rows = sorted worker * b + sample).
struct Workspace {
  float* p1;       // conv1 -> ReLU -> pool: [rows][16][14][14] fp32 (FP32 path) or [rows][2 planes][256][8] BF16 (tensor-core path)
  uint8_t* code1;  // [rows][3136]        pool-1 decisions. FP32 path: [16][196], argmax 0..3, 4 = no gradient (max <= 0); tensor-core path:
                   //                     [4 channel quads][196][4], the byte 1 << argmax, 0 = no gradient
  float* p2;       // [rows][1568]        conv2 -> ReLU -> pool, channel-major flatten
  uint8_t* code2;  // [rows][1568]
  float* d;        // [rows][512]         fc1 -> ReLU -> dropout (scaled)
  float* da1;      // [rows][512]         gradient w.r.t. fc1 pre-activation
  float* dz;       // [rows][16]          gradient w.r.t. logits (10 used)
  float* dp2;      // [rows][1568]        gradient w.r.t. p2 (tensor-core path: BF16 in the first half of each row)
  float* dp1;      // [rows][3136]        gradient w.r.t. p1; [16][196] fp32 (FP32 path) or [4 channel quads][196][4] BF16 in the first half of the row (tensor-core path)
  float* part2;    // [W][chunks][4640]   per-block partial conv2 weight/bias gradients
  float* part1;    // [W][8 chunks][160]  per-block partial conv1 weight/bias gradients (tensor-core path: eight per range, one per sample of a pair and window element)
  float* partf;    // [W][FC2_SPLIT][FC_PART] per-block partial output-layer gradients and loss sums
  float* w1r;      // [groups][512][1568] TF32-rounded fc1 weights of each weight group of the call
  float* w1tr;     // [groups][1568][512] and their transpose
  uint32_t* status;
};

struct GradStepArgs {
  int W, b;
  const float* x;      // [W][b][784] caller order
  const int32_t* y;    // [W][b]
  float* loss;         // [W]
  int32_t* argmax;     // [W][b]
  uint64_t seed, step;
  float drop_p;
  uint32_t drop_thresh;   // keep iff word >= thresh
  int precision;          // 0 = FP32 CUDA cores; otherwise tensor cores (BF16 convolution products, TF32 dense layer)
  int skip_prep_w1;       // the rounded copies of the dense-layer weights of these very snapshots are still valid
};

// Side streams (and the events that fork from / join into the caller's stream) for the independent
// branches of the backward pass; null streams mean "run everything on the caller's stream".
struct SideStreams {
  cudaStream_t s1 = nullptr, s2 = nullptr;
  cudaEvent_t fork1 = nullptr, join1 = nullptr, fork2 = nullptr, join2 = nullptr;
};

// The summed step (all workers on one snapshot, only the sum of their gradients wanted): where it goes and the scratch
// for the partial sums of the 512-unit layer's weight gradient.
struct SummedStep {
  float* grad_sum;      // [P_PAD] the sum over workers
  float* super_part;    // [n_super][P_PAD] scratch
  int n_super;          // groups of W / n_super workers (a divisor of W, at most 16)
};

// Part A. Returns the number of kernels launched, or -1 on a launch error.  sum == nullptr: one gradient per worker.
int launch_grad_step(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                     cudaStream_t st, const SideStreams& side, Profiler* prof, const SummedStep* sum = nullptr);
int launch_dropout_mask(uint64_t seed, uint32_t worker, uint64_t step, int b, uint32_t thresh,
                        uint8_t* keep, cudaStream_t st, Profiler* prof);
int configure_grad_kernels();
extern int g_sm_count;   // SMs of the current device, set by configure_tc5_kernels
int configure_tc5_kernels();
int configure_conv5_kernels();
int configure_conv1_kernels();
int configure_dw5_kernels();
int configure_c1d5_kernels();
int launch_conv1_dw_tc5(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof,
                        int* seg_len);
int launch_conv2_dw_tc5(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof,
                        int* seg_len);
int launch_conv1_fwd_planes(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                            cudaStream_t st, Profiler* prof);
void launch_conv2_fwd_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                          cudaStream_t st, Profiler* prof);
void launch_conv2_dx_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                         cudaStream_t st, Profiler* prof);
int launch_prep_w1(const GroupTable& gt, const Workspace& ws, cudaStream_t st, Profiler* prof);
int launch_fc1_fwd_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                       cudaStream_t st, Profiler* prof);
int launch_fc1_dx_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                      cudaStream_t st, Profiler* prof);
int launch_fc1_dw_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                      cudaStream_t st, Profiler* prof);

// Part B.
struct SumApplyArgs {
  const float* queue;       // slot 0 of the gradient queue; slot k at queue + k*P_PAD
  int64_t K;                // gradients to sum (slots 0..K-1)
  const float* theta_in;    // current head
  float* theta_out;         // new head (may equal theta_in)
  float* replica;           // mirror target or nullptr
  float coef;               // lr*scale/divisor
  float* partial;           // [max_split][P_PAD] scratch
  int max_split;
  const float* coef_k;      // per-gradient factors [K] that replace coef (the stale-gradient treatments), or nullptr
};
int launch_sum_apply(const SumApplyArgs& a, cudaStream_t st, Profiler* prof);

constexpr int ASYNC_SEG = 256;   // gradients per ordered-apply launch
struct AsyncOrder { int32_t slot[ASYNC_SEG]; };
struct AsyncApplyArgs {
  const float* queue;
  int K;                    // 1..ASYNC_SEG gradients in this segment
  const float* theta_in;    // version v0
  float* ring[MAX_RING];    // ring slot buffers
  int ring_depth;
  uint64_t v0;              // version of theta_in; version v0+k+1 is stored in ring[(v0+k+1) % depth]
  int first_stored;         // only k >= first_stored are stored (the last ring_depth versions)
  int n_mirror;             // chain-replication stores of this segment (at most one per server behind the frontend)
  int mirror_k[MAX_CHAIN];  // k whose result is also written to replica[m]
  float* replica[MAX_CHAIN];
  float coef;               // lr*scale
  const float* coef_k;      // per-gradient factors indexed by queue slot that replace coef, or nullptr
};
int launch_async_apply(const AsyncApplyArgs& a, const AsyncOrder& ord, cudaStream_t st, Profiler* prof);

int launch_copy_rows(float* dst, const float* src, int64_t rows, cudaStream_t st, Profiler* prof);

// Clipping by global norm: coef_k[k] *= min(1, clip / ||queue[k]||_2) for k < K.  norm_part: [K][NORM_CHUNKS] scratch.
constexpr int NORM_CHUNKS = 8;
int launch_clip_factors(const float* queue, int64_t K, float clip, float* coef_k, float* norm_part, cudaStream_t st, Profiler* prof);

// Evaluation pass: forward only, no dropout; loss [W] mean cross-entropy, argmax [W][b], correct [W] = samples whose
// argmax equals the label.  Returns the number of kernels launched or -1.
int launch_eval(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws, int32_t* correct,
                cudaStream_t st, Profiler* prof);

// One warp waits on a barrier nobody arrives at, for at most limit_cycles, then sets STATUS_WAIT_TIMEOUT in *status.
int launch_wait_timeout_probe(uint32_t* status, long long limit_cycles, cudaStream_t st);

}  // namespace psk
