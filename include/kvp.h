/* kvp.h -- C ABI of the B200 shared-KV attention library (KV-Pipe hot path).
 *
 * The library implements the attention block of a decoder stack in which KV-sharing
 * ("consumer") layers keep only their query projection and attend to the keys/values of an
 * earlier "donor" layer (Eq. 3 of the paper: K_l <- K_tau(l), V_l <- V_tau(l), tau(l) < l),
 * plus the paper's offline planner (Algorithm 1) that decides which layers to convert.
 *
 * Conventions for every entry point
 *  - Returns an int status (KVP_OK == 0).  No exceptions, no allocation, no host
 *    synchronisation in the device entry points: all device work is enqueued on the caller's
 *    stream and the caller owns every buffer (inputs, outputs, workspace, cache, tables).
 *  - "device" pointers must be 16-byte aligned device memory; "host" pointers are host memory.
 *  - Per-layer tensors are passed as HOST arrays of length L holding DEVICE pointers.  Entries
 *    of K/V-like arrays are read only for owner layers (donor[l] == l) and may be NULL elsewhere.
 *  - donor is a HOST int32[L] with donor[l] <= l and donor[donor[l]] == donor[l]; anything else
 *    returns KVP_ERR_BAD_DONOR.
 *  - Activations are [B, S, H, dh] (token-major, dh contiguous); weights are [out, in]
 *    row-major; LSE is [B, Hq, S] fp32, the natural log of the row sum of exp(scaled scores).
 *  - Query head hq reads KV head hq / (Hq / Hkv) (contiguous GQA groups).
 *  - dtype KVP_BF16: X, W, Q, K, V, O, dO, dQ, dX, Y are bf16 (round-to-nearest-even where
 *    the library stores them); LSE, dK/dV sums and all weight gradients are fp32; all
 *    accumulation is fp32.
 *  - dtype KVP_F32 (the tiny-stack configuration's "fp32"): the same tensors are fp32 in the caller's memory.  The
 *    library converts them on load to bf16 (round-to-nearest-even; values that are bf16-representable pass
 *    unchanged) and widens its bf16 results on store, so the arithmetic, and the results, are those of KVP_BF16:
 *    one code path.  The training entry points then keep the bf16 copies in the workspace (kvp_workspace_bytes
 *    accounts for them, also for KVP_OP_PROJ_FWD / KVP_OP_ATTN_FWD, which need none otherwise); the decode entry
 *    points read fp32 queries / new K, V rows and write fp32 outputs directly (the cache itself stays bf16).
 *    kvp_out_proj_* and kvp_gemm take bf16 only.
 *  - Supported: dh in {64, 128}; Hq % Hkv == 0; D % 64 == 0; S >= 1.  Anything else returns
 *    KVP_ERR_UNSUPPORTED -- there is no slow path and no CPU fallback.
 *  - Kernels that wait on hardware barriers give up after about two seconds, record
 *    KVP_ERR_TIMEOUT in a device status word and exit cleanly; kvp_device_status() reads it.
 */
#ifndef KVP_H_
#define KVP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* kvp_stream_t; /* a cudaStream_t */

enum {
  KVP_OK = 0,
  KVP_ERR_INVALID_ARG = 1,
  KVP_ERR_BAD_DONOR = 2,
  KVP_ERR_UNSUPPORTED = 3,
  KVP_ERR_WORKSPACE = 4,
  KVP_ERR_CUDA = 5,
  KVP_ERR_TIMEOUT = 6
};

enum { KVP_BF16 = 0, KVP_F32 = 1 };

/* Returns a static string for a status code. */
const char* kvp_status_string(int status);

/* Synchronises the device and returns KVP_OK, or KVP_ERR_TIMEOUT if any kernel of this library
 * gave up on a bounded wait since the last call (the word is cleared), or KVP_ERR_CUDA. */
int kvp_device_status(void);

/* Self-test of the bounded waits (the library's failure detection; the paper has no counterpart).  Enqueues one
 * small GEMM in which the MMA-issuing warp withholds, once, the barrier arrival that frees a shared-memory ring
 * stage, with a wait limit of 5 ms instead of two seconds: the TMA warp's wait for that stage runs out, it records
 * the timeout, every other role sees the flag at its own next wait, and the kernel frees its TMEM and exits.  The
 * call returns KVP_OK once the launch is enqueued; afterwards kvp_device_status() must return KVP_ERR_TIMEOUT
 * (once: the word is cleared) and the device and the library remain usable.  Nothing faults and nothing spins
 * without a limit.  scratch: DEVICE memory, 16-byte aligned, at least 512 KiB, contents irrelevant and clobbered. */
int kvp_selftest_bounded_wait(void* scratch, size_t scratch_bytes, kvp_stream_t stream);
/* The same self-test on the CTA-pair GEMM kernel (one 256 x 256 tile on a cluster of two CTAs): the issuing CTA
 * withholds, once, the arrivals that free a ring stage in both CTAs; both producers' waits run out, every role of
 * both CTAs falls through to the common teardown (the two CTAs wait for each other, then free their TMEM).
 * scratch: at least 768 KiB.  Refused with KVP_ERR_UNSUPPORTED while kvp_set_gemm_pair_mode(0) is in force. */
int kvp_selftest_bounded_wait_pair(void* scratch, size_t scratch_bytes, kvp_stream_t stream);

/* Benchmark bookkeeping.  kvp_launch_count: kernels launched by this library since it was loaded.
 * kvp_set_timing_events: record the caller's CUDA events (HOST arrays of n cudaEvent_t, created by
 * the caller) immediately before and after each of the next n launches of one kernel
 * (0 GEMM, 1 attention forward, 2 attention backward, 3 decode, 4 the backward's helper passes: Delta, accumulator clear, dQ conversion, one pair per group of launches); n == 0 switches it off.
 * kvp_timing_events_used: how many pairs have been recorded since.  Not thread-safe. */
unsigned long long kvp_launch_count(void);
int kvp_set_timing_events(int kernel, void** starts, void** stops, int n);
int kvp_timing_events_used(int kernel);
/* Measurement switch of the GEMM's tile shape.  1 (the default): the forward GEMMs (kvp_proj_fwd,
 * kvp_out_proj_fwd, kvp_gemm) run on CTA pairs (256 x 256 tiles, one per pair of SMs) when every problem of the
 * launch has more than 128 rows, the gradient GEMMs on single-CTA 128 x 256 tiles; 0: single-CTA tiles
 * everywhere; 2: CTA pairs everywhere.  The results are the same in every mode (same products, same summation
 * order along K).  Not thread-safe. */
void kvp_set_gemm_pair_mode(int mode);

/* ------------------------------------------------------------------------------------------
 * Planner (host only, pure, exact integer arithmetic).
 *
 * kvp_plan is Algorithm 1 of the paper ("KV-Pipe (Architecture-Balanced)"): starting from the
 * last pipeline stage it converts the deepest unconverted layer of the chosen stage to KV
 * sharing, retargets to the arg-max stage once the tail is within (1+eps) of the average, and
 * stops when FIR <= 1+eps (Eq. 4-5), when the budget is spent, or when the chosen stage has no
 * convertible layer.  FIR is kept as the exact fraction fir_num / fir_den = max_i F_i * P / sum F.
 *
 * Readings where the paper is silent: tau(l) is the nearest preceding unconverted layer; layer 0
 * is never converted; arg-max ties go to the highest stage index; KVP_PLAN_STOP_ON_NO_IMPROVE
 * rejects (and stops at) a conversion that would not strictly lower FIR; KVP_PLAN_STAGE_LOCAL_DONOR
 * keeps the first layer of every stage unconverted; alpha (appendix "Optional Safe-Layer
 * Guardrail") admits only layers with 1-indexed l >= ceil(alpha L).
 * ---------------------------------------------------------------------------------------- */
enum { KVP_PLAN_STOP_ON_NO_IMPROVE = 1, KVP_PLAN_STAGE_LOCAL_DONOR = 2 };
enum { KVP_STOP_TOLERANCE = 0, KVP_STOP_BUDGET = 1, KVP_STOP_EXHAUSTED = 2, KVP_STOP_NO_IMPROVE = 3 };
enum { KVP_PLACE_ARCH_BALANCED = 0, KVP_PLACE_UNIFORM = 1, KVP_PLACE_BIPOLAR = 2 };

typedef struct {
  int32_t L;                    /* layers */
  int32_t P;                    /* pipeline stages */
  const int32_t* stage_begin;   /* host [P+1], stage i holds layers stage_begin[i] .. stage_begin[i+1]-1 */
  const uint64_t* f_full;       /* host [L], cost of layer l with full attention, F_l(0) */
  const uint64_t* f_share;      /* host [L], cost with KV sharing, F_l(1) < F_l(0) */
  const uint64_t* stage_extra;  /* host [P], non-layer cost per stage (LM head on the last stage) */
  uint32_t eps_num, eps_den;    /* tolerance eps = eps_num / eps_den (eps_den > 0) */
  int32_t max_conv;             /* budget m; 0 means L */
  uint32_t flags;               /* KVP_PLAN_* */
  uint32_t alpha_num, alpha_den;/* guardrail alpha; alpha_num == 0 disables it */
  int32_t placement;            /* KVP_PLACE_*; UNIFORM / BIPOLAR place exactly max_conv layers */
} kvp_plan_in;

typedef struct {
  uint8_t* z;             /* host [L] out: 1 = converted to KV sharing */
  int32_t* donor;         /* host [L] out: tau(l) */
  uint64_t* stage_flops;  /* host [P] out: F_stage_i(z), Eq. 6 */
  double* stage_ratio;    /* host [P] out: F_i * P / sum F */
  uint64_t fir_num;       /* max_i F_i * P */
  uint64_t fir_den;       /* sum_i F_i */
  double fir;             /* (double)fir_num / (double)fir_den */
  int32_t n_conv;
  int32_t stop_reason;    /* KVP_STOP_* */
} kvp_plan_out;

int kvp_plan(const kvp_plan_in* in, kvp_plan_out* out);

/* Analytic per-token forward FLOPs of one decoder layer (appendix "Attention FLOPs under MHA and
 * GQA", a MAC counted as 2): Q and output projections 2*h*(a*dh) each, K and V projections
 * 2*h*(g*dh) each, scores and weighted sum 2*s*(a*dh) each (halved when causal_half != 0 -- the
 * count that reproduces the paper's printed FIR), gated MLP 6*h*f.  f_share = f_full minus the K/V
 * projections (the paper's Delta F = 4 h^2 / r); f_lm_head = 2*h*vocab. */
typedef struct {
  int32_t h, f, a, g, dh, s, vocab, causal_half;
} kvp_model_desc;
int kvp_layer_flops(const kvp_model_desc* m, uint64_t* f_full, uint64_t* f_share, uint64_t* f_lm_head);

/* 1F1B pipeline timing model (host only, pure, exact integer arithmetic).
 *
 * The paper measures KV-Pipe under the non-interleaved 1F1B schedule (section "Results on Ascend
 * 910B NPUs") and ties the iteration time to the stage imbalance FIR (Eq. 4-5); it prints no timing
 * model.  kvp_sim_1f1b evaluates that schedule for given per-stage times: stage i of P runs
 * min(P-1-i, M) warm-up forwards, then alternates one forward and one backward, then drains its
 * remaining backwards, strictly in that order; forward (i, m) needs forward (i-1, m), backward (i, m)
 * needs backward (i+1, m) (its own forward on the last stage); transfers cost nothing.  An operation
 * starts when its inputs exist and the stage is free.
 *
 * t_fwd / t_bwd: host [P], time of one micro-batch on stage i, any unit, >= 0.  out->makespan is the
 * finish time of the last operation; out->idle (host [P], may be NULL) receives
 * makespan - M * (t_fwd[i] + t_bwd[i]), the stage's bubble.  P >= 1, M >= 1 and P * M <= 2^24, else
 * KVP_ERR_INVALID_ARG.  Feeding measured stage times of a converted and an unconverted stage gives the
 * iteration-time effect of a plan without a multi-device run. */
typedef struct {
  int64_t makespan;
  int64_t* idle;
} kvp_sim_out;
int kvp_sim_1f1b(int32_t P, int32_t M, const int64_t* t_fwd, const int64_t* t_bwd, kvp_sim_out* out);

/* ------------------------------------------------------------------------------------------
 * Training / prefill path
 * ---------------------------------------------------------------------------------------- */
typedef struct {
  int32_t L, B, S, D, Hq, Hkv, dh;
  int32_t dtype; /* KVP_BF16 or KVP_F32 */
} kvp_shape;

enum { KVP_OP_PROJ_FWD = 0, KVP_OP_PROJ_BWD = 1, KVP_OP_ATTN_FWD = 2, KVP_OP_ATTN_BWD = 3, KVP_OP_DECODE = 4 };

/* Bytes of device workspace an op needs for this shape (decode: pass the kvp_decode_desc through
 * kvp_decode_workspace_bytes instead).  0 is a valid answer. */
size_t kvp_workspace_bytes(int op, const kvp_shape* s, const int32_t* donor);

/* Eq. 1.  q[l] = x[l] wq[l]^T for every layer; k[l] = x[l] wk[l]^T, v[l] = x[l] wv[l]^T for owners
 * only (Eq. 3 removes them for consumers).  x[l]: [B*S, D]; wq[l]: [Hq*dh, D]; wk[l], wv[l]:
 * [Hkv*dh, D]; q[l]: [B,S,Hq,dh]; k[l], v[l]: [B,S,Hkv,dh].  All projections of all layers are tiles of one
 * grouped GEMM launch (one launch per 32 projections). */
int kvp_proj_fwd(const kvp_shape* s, const int32_t* donor, const void* const* x, const void* const* wq,
                 const void* const* wk, const void* const* wv, void* const* q, void* const* k, void* const* v,
                 void* ws, size_t ws_bytes, kvp_stream_t stream);

/* Chain rule of Eq. 1.  dwq[l] = dq[l]^T x[l] (fp32 [Hq*dh, D]); dx[l] = dq[l] wq[l] (bf16 [B*S, D]);
 * owners add dwk = dk_sum^T x, dwv = dv_sum^T x and dx += dk_sum wk + dv_sum wv, where dk_sum, dv_sum
 * (fp32 [B,S,Hkv,dh]) are the donor-group sums written by kvp_attn_bwd, rounded once to bf16.
 * Layers are taken eight at a time: the sums of the eight layers' owners are rounded into the workspace, then one
 * grouped GEMM launch writes every gradient of those layers.
 * Workspace: kvp_workspace_bytes(KVP_OP_PROJ_BWD, ...) = bf16 copies of dk_sum and dv_sum for min(owners, 8) layers. */
int kvp_proj_bwd(const kvp_shape* s, const int32_t* donor, const void* const* x, const void* const* wq,
                 const void* const* wk, const void* const* wv, const void* const* dq, const float* const* dk_sum,
                 const float* const* dv_sum, float* const* dwq, float* const* dwk, float* const* dwv,
                 void* const* dx, void* ws, size_t ws_bytes, kvp_stream_t stream);

/* kvp_proj_bwd restricted to layers layer_begin <= l < layer_end (same arrays of length L, same workspace): lets a
 * data-parallel caller start the cross-rank sum of one layer's weight gradients while the next layer's are still
 * being computed.  KVP_BF16 only. */
int kvp_proj_bwd_range(const kvp_shape* s, const int32_t* donor, const void* const* x, const void* const* wq,
                       const void* const* wk, const void* const* wv, const void* const* dq, const float* const* dk_sum,
                       const float* const* dv_sum, float* const* dwq, float* const* dwk, float* const* dwv,
                       void* const* dx, int layer_begin, int layer_end, void* ws, size_t ws_bytes, kvp_stream_t stream);

/* Output projection y[l] = o[l] wo[l]^T and its chain rule (d_o = dy wo, dwo = dy^T o); the paper's
 * 2bsh^2 "output projection" term.  o[l]: [B*S, Hq*dh]; wo[l]: [D, Hq*dh]; y[l]: [B*S, D]. */
int kvp_out_proj_fwd(const kvp_shape* s, const void* const* o, const void* const* wo, void* const* y,
                     kvp_stream_t stream);
int kvp_out_proj_bwd(const kvp_shape* s, const void* const* o, const void* const* wo, const void* const* dy,
                     void* const* d_o, float* const* dwo, kvp_stream_t stream);

/* Eq. 2-3.  o[l] = softmax(q[l] k[d]^T * scale + M) v[d] with d = donor[l], M the causal mask when
 * causal != 0 (key j visible to query i iff j <= i); scale == 0 means 1/sqrt(dh).
 * o[l]: [B,S,Hq,dh] bf16; lse[l]: [B,Hq,S] fp32.  Up to eight layers run as one launch of persistent CTAs. */
int kvp_attn_fwd(const kvp_shape* s, const int32_t* donor, int causal, float scale, const void* const* q,
                 const void* const* k, const void* const* v, void* const* o, float* const* lse, void* ws,
                 size_t ws_bytes, kvp_stream_t stream);

/* Chain rule of Eq. 2-3.  dq[l] (bf16) per layer; dk_sum[d], dv_sum[d] (fp32 [B,S,Hkv,dh], owners
 * only) are the sums over the donor, all its consumers and the Hq/Hkv query heads of each KV head,
 * accumulated in fp32 on chip across layers, heads and query tiles.  The scores are computed once per
 * tile pair for all three gradients; partial sums that different thread blocks own (dq over key tiles, dk_sum /
 * dv_sum over windows of query tiles) are combined by fp32 reductions in global memory, so these outputs are
 * reproducible up to fp32 summation order, not bit for bit.  dk_sum / dv_sum are overwritten (cleared first),
 * never accumulated into.  At most 8 layers may share one donor.
 * Workspace: kvp_workspace_bytes(KVP_OP_ATTN_BWD): Delta per layer plus fp32 dq accumulators for up to 8 layers. */
int kvp_attn_bwd(const kvp_shape* s, const int32_t* donor, int causal, float scale, const void* const* q,
                 const void* const* k, const void* const* v, const void* const* o, const void* const* d_o,
                 const float* const* lse, void* const* dq, float* const* dk_sum, float* const* dv_sum, void* ws,
                 size_t ws_bytes, kvp_stream_t stream);

/* Building block of the projections: C[M,N] = A B, bf16 inputs, fp32 accumulate.
 * a_mn == 0: A stored [M,K] row-major, else stored [K,M].  b_mn == 0: B stored [N,K] row-major
 * (C = A B^T in storage terms), else stored [K,N].  out_f32: C fp32, else bf16.  Leading dimensions
 * in elements, multiples of 8; K a multiple of 8.  The paper's 2mkn matrix-multiplication rule. */
int kvp_gemm(int M, int N, int K, const void* a, int64_t lda, int a_mn, const void* b, int64_t ldb, int b_mn,
             void* c, int64_t ldc, int out_f32, kvp_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * Element-wise operators of a decoder stage.
 *
 * The paper's stage tables list a forward time per pipeline stage of LLaMA2-7B but define no operator
 * besides attention (Eq. 1-3); these are the published definitions of the architecture it names, provided
 * so that a whole stage's forward pass can be timed with this library.  Device pointers, 16-byte aligned,
 * bf16 storage, fp32 arithmetic, asynchronous on `stream`; `out` may alias an input.
 *   kvp_rmsnorm  y[T,D] = x / sqrt(mean_D(x^2) + eps) * w[D]; D a multiple of 8, D <= 8192.
 *   kvp_rope     in place on x [B,S,H,dh]: consecutive pairs (x[2i], x[2i+1]) of every head are rotated by
 *                (pos0 + s) * theta^(-2i/dh); dh a multiple of 8, dh <= 256, pos0 + S <= 2^18.
 *   kvp_swiglu   out[n] = silu(gate) * up, silu(t) = t / (1 + exp(-t)); n a multiple of 8.
 *   kvp_add      out[n] = a + b; n a multiple of 8.
 * KVP_ERR_INVALID_ARG for null pointers / negative sizes, KVP_ERR_UNSUPPORTED for the shape limits.
 * ---------------------------------------------------------------------------------------- */
int kvp_rmsnorm(int32_t T, int32_t D, const void* x, const void* w, float eps, void* y, kvp_stream_t stream);
int kvp_rope(int32_t B, int32_t S, int32_t H, int32_t dh, float theta, int32_t pos0, void* x, kvp_stream_t stream);
int kvp_swiglu(int64_t n, const void* gate, const void* up, void* out, kvp_stream_t stream);
int kvp_add(int64_t n, const void* a, const void* b, void* out, kvp_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * Decode over the shared paged cache
 * ---------------------------------------------------------------------------------------- */
typedef struct {
  int32_t L, B, Hq, Hkv, dh;
  int32_t page_size;  /* tokens per page: a multiple of 16 */
  int32_t max_pages;  /* columns of block_table */
  int32_t n_pages;    /* pages in each owner layer's pool */
  int32_t num_splits; /* KV splits per (sequence, KV head); 0 lets the library choose */
  int32_t dtype;      /* KVP_BF16, or KVP_F32: q, k_new, v_new, o are fp32; the cache is bf16 either way */
} kvp_decode_desc;

size_t kvp_decode_workspace_bytes(const kvp_decode_desc* d, const int32_t* donor);

/* "Each layer appends (K_l, V_l) into the KV cache": owners write k_new[l][b], v_new[l][b]
 * ([B,Hkv,dh]) at position lengths[b]-1 of sequence b; consumers store nothing.
 * k_cache[l], v_cache[l]: page pools [n_pages][Hkv][page_size][dh] (owners only).
 * block_table: DEVICE int32 [B, max_pages], page of sequence b holding positions
 * [i*page_size, (i+1)*page_size).  lengths: DEVICE int32 [B], length INCLUDING the new token. */
int kvp_cache_append(const kvp_decode_desc* d, const int32_t* donor, const void* const* k_new,
                     const void* const* v_new, void* const* k_cache, void* const* v_cache,
                     const int32_t* block_table, const int32_t* lengths, kvp_stream_t stream);

/* o[l][b,hq] = softmax(q[l][b,hq] . K_d[b, 0:len]^T * scale) V_d[b, 0:len] over the donor's pages
 * for layers layer_begin <= l < layer_end.  A donor and its consumers inside the range are served
 * by one pass over the donor's pages (each page read once per donor, not once per layer) as long as
 * the group's query rows fit one pass: min(4, 16 / (Hq/Hkv)) layers; a larger group takes one pass
 * per that many layers.
 * q[l], o[l]: [B,Hq,dh] bf16; lse[l]: [B,Hq] fp32.  lengths outside [1, max_pages*page_size] are
 * clamped.  Workspace: kvp_decode_workspace_bytes. */
int kvp_decode(const kvp_decode_desc* d, const int32_t* donor, float scale, const void* const* q,
               const void* const* k_cache, const void* const* v_cache, const int32_t* block_table,
               const int32_t* lengths, void* const* o, float* const* lse, int layer_begin, int layer_end, void* ws,
               size_t ws_bytes, kvp_stream_t stream);

/* kvp_decode without a workspace argument and without any allocation (the paper has no counterpart:
 * this is a packaging variant of kvp_decode, same arithmetic, same outputs).
 *
 * For callers that cannot obtain device memory where they decode -- a serving loop that has given
 * the whole device to its cache pool, a plug-in whose host forbids cudaMalloc on its hot path, a
 * worker that must stay out of the allocator.  The per-split partial results are kept in an array
 * of KVP_DECODE_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads the
 * library holds those bytes until the process exits.
 *
 *  - A request whose partials need more than that (they grow with the number of donor groups that
 *    [layer_begin, layer_end) touches, up to 64 per launch, and with B, Hkv and the split count;
 *    kvp_decode_workspace_bytes(d, donor) is the figure for all layers) is refused with
 *    KVP_ERR_STATIC_SCRATCH and nothing is launched; lower num_splits, decode a narrower layer
 *    range per call, or use kvp_decode with your own workspace.
 *  - No cudaMalloc / cudaFree / allocating library call is made, on any call.
 *  - The first call on each device looks up the array's device address (with that device current);
 *    make that first call outside any stream capture.
 *  - The array is shared by every call and keeps the previous call's contents.  Nothing in it has to
 *    start at zero: each partial is written by the decode kernel before the combine kernel reads it.
 *    Two calls whose kernels overlap on the GPU (different streams, or different host threads) race
 *    on it and corrupt each other's results; serialise them on one stream.
 *  - All other arguments, layouts and status codes are those of kvp_decode. */
#define KVP_DECODE_STATIC_SCRATCH_BYTES (16u << 20)
enum { KVP_ERR_STATIC_SCRATCH = 7 };
int kvp_decode_static(const kvp_decode_desc* d, const int32_t* donor, float scale, const void* const* q,
                      const void* const* k_cache, const void* const* v_cache, const int32_t* block_table,
                      const int32_t* lengths, void* const* o, float* const* lse, int layer_begin, int layer_end,
                      kvp_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* KVP_H_ */
