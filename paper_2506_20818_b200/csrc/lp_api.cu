// C ABI of the link-prediction training step: context, validation, workspace and the
// orchestration of the kernels.  See include/lp.h for the contract of every entry point.
#include <algorithm>
#include <cmath>
#include <memory>
#include <new>

#include "common.cuh"
#include "scan_sort.cuh"
#include "spmm.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "sampler.cuh"
#include "edge.cuh"
#include "optim.cuh"
#include "sparsify.cuh"
#include "view.cuh"
#include "predictor.cuh"
#include "probe.cuh"

// ----------------------------------------------------------------------------------------------
// context
// ----------------------------------------------------------------------------------------------
struct HopBlock {  // sampled block of hop h (destinations F_{h-1}, sources F_h)
    int cap_dst = 0, cap_src = 0;
    int64_t cap_entries = 0;
    int n_dst = 0, n_src = 0;  // host mirrors of the last step
    int64_t entries = 0;
    int *frontier = nullptr;      // F_h, global ids ascending            [cap_src]
    int *n_front_dev = nullptr;   // |F_h| on the device
    int *posmap = nullptr;        // global id -> position in F_h          [n]
    int *blk_ptr = nullptr;       // offsets per destination               [cap_dst + 1]
    int *blk_col_global = nullptr, *blk_col_local = nullptr, *blk_row = nullptr;  // [cap_entries]
    float *inv_deg = nullptr;     // 1 / sampled degree per destination     [cap_dst]
    int *colptr = nullptr, *rowidx = nullptr, *perm = nullptr;  // transposed block
    int *self_idx = nullptr, *inv_self = nullptr;
    // GCN only: CSR position of every sampled entry, its rescaled coefficient (block order and transposed
    // order) and the self coefficients 1 / d~ of the destination and of the source rows
    int *blk_eid = nullptr;
    float *blk_val = nullptr, *blk_valT = nullptr, *self_coef_dst = nullptr, *self_coef_src = nullptr;
};

struct LayerBuf {  // device buffers of one encoder layer (element type fixed by the precision)
    void *A = nullptr;     // GEMM operand: SAGE [rows, 2 Fi] = [H | mean]; GCN [rows, Fi] = aggregate
    void *Hin = nullptr;   // input embeddings H^(k) when they are not the left half of A
    void *Hout = nullptr;  // sampled models: output rows of this layer [rows_dst, Fo]
    int64_t off_w = 0, off_b = 0;  // offsets in the flat parameter vector
    int Fi = 0, Fo = 0, Kin = 0;
};

struct lp_ctx {
    int device = 0;
    Exec ex;
    std::string err;
    std::vector<void *> graph_allocs, model_allocs, sparse_allocs;
    int64_t graph_bytes = 0, model_bytes = 0, sparse_bytes = 0;
    int64_t *sp_ptr = nullptr;  // last sparsified graph
    int *sp_col = nullptr;
    float *sp_w = nullptr;
    int64_t sp_nnz = -1;
    std::vector<void *> view_allocs;
    int64_t view_bytes = 0, view_nnz = -1;
    int *view_ptr = nullptr, *view_col = nullptr;  // last worker view

    // graph
    bool loaded = false;
    int n = 0, f = 0;
    int64_t nnz = 0;
    int *rowptr = nullptr, *col = nullptr;
    float *w = nullptr;
    int *colptr = nullptr, *rowidx = nullptr, *perm = nullptr;
    float *gcn_val = nullptr, *gcn_valT = nullptr, *gcn_self = nullptr;
    float *inv_deg = nullptr, *meanT_val = nullptr;
    float *X32 = nullptr;
    bf16 *X16 = nullptr;
    int *cand = nullptr;         // candidate set of the negative sampler (own allocation, replaced by every lp_set_candidates)
    int64_t n_cand = 0;
    unsigned long long *exhausted_dev = nullptr;  // 16 counters used in turn: a call of the sampler adds into one and clears the next
    uint64_t neg_calls = 0;
    HeavyPlan plan_csr, plan_csc, plan_dyn;  // heavy-row plans: the loaded graph, its transpose, per-step structures
    float *heavy_partials = nullptr;
    int *err_flag = nullptr;

    // model
    bool model_set = false, sampled = false;
    lp_model_desc desc{};
    int64_t n_params = 0, max_batch = 0;
    int max_k = 0, K = 0;
    LayerBuf layer[LP_MAX_LAYERS];
    void *HK = nullptr;                 // H^(K) [rows_out, D]
    int64_t inc_cap = 0;                // ints in inc_ptr
    void *dHK = nullptr;                // dL/dH^(K) [rows_out, D]
    void *dZ[2] = {nullptr, nullptr};   // gradient ping-pong [max_rows, max_width]
    void *dA = nullptr;                 // [max_rows, max Kin]
    float *partials = nullptr;          // split-K / column-sum partials
    int64_t partials_floats = 0;
    float *g_pos = nullptr, *g_neg = nullptr, *loss_partials = nullptr;
    // MLP edge predictor
    bool mlp = false;
    int Hp = 0;
    int64_t n_enc_params = 0;           // parameters of the encoder; the predictor's follow
    int64_t off_w2 = 0, off_b2 = 0;
    LayerBuf pred[2];                   // the two wide predictor layers (A = Z0, then P1)
    void *P2 = nullptr, *dPa = nullptr, *dPb = nullptr, *dZ0 = nullptr;
    float *pred_scores = nullptr;       // [E]
    int *inc_edge = nullptr;            // edge of every incidence entry (row of dL/dz0)
    int *inc_cursor = nullptr, *inc_ptr = nullptr, *inc_col = nullptr;
    float *inc_partials = nullptr;      // 64-bit item partials of the exact gather over the incidence lists
    float *inc_val = nullptr;
    SortScratch sort;                   // sized for the largest per-step sort
    TransposeScratch tsp;
    int *scan_tmp = nullptr;
    OnePassScan scan1;                  // single-launch scan of the step's per-node counts
    int64_t sort_cap = 0;
    HopBlock hop[LP_MAX_LAYERS + 1];    // hop[0] holds only the seed frontier F_0
    unsigned char *mark = nullptr;
    int *flags = nullptr;
    int *seed_ids = nullptr;            // pos_src | pos_dst | neg_dst (| neg_src) of the batch
    int *host_counts = nullptr;         // pinned
    int *d_neg_tmp = nullptr, *d_pos_tmp = nullptr;  // staging of lp_train_step_host
    float *d_loss_tmp = nullptr, *d_grads_tmp = nullptr;
    int rows_out = 0;                   // rows of H^(K) in the last forward
    bool have_forward = false, have_grad = false;
    bool input_agg_valid = false;       // cached AGG(X) of layer 1 is present (cache_input_aggregation)
    // H^(K) of the last full-graph forward pass stays valid for lp_score while the same parameter vector is passed and no
    // call of this library has changed it (param_version counts such calls)
    bool hk_valid = false;
    const float *hk_params = nullptr;
    uint64_t hk_version = 0, param_version = 0;
    int64_t last_exhausted = 0;
    TcState tc;                         // tensor-core GEMM state (descriptor encoder, device error word)
    bf16 *w16 = nullptr, *w16t = nullptr;  // BF16 path: the parameter vector of the current call as BF16, as is and with every weight matrix transposed
    bf16 *w16s = nullptr;                  // ... and with the SAGE layers' [W_self ; W_neigh] stored side by side (see weights_cache_kernel)
    // One-pass SAGE layers l >= 1 on the tensor-core pair kernel take the input gradient as
    // dH^(l) = relu'(H^(l)) * ([dZ | A^T dZ / deg] [W_self^T ; W_neigh^T]): the adjoint aggregation runs on dZ (no self term, no mask),
    // the transform reads the two halves side by side and applies the ReLU mask from sign-bit words the forward transform left.
    bool cat_grad[LP_MAX_LAYERS] = {};
    uint32_t *relu_bits[LP_MAX_LAYERS] = {};  // [Fi / 32][n] words of layer l's input H^(l)
    void *dcat[2] = {nullptr, nullptr};       // [n, 2 * max Fo] gradient operands (dZ | adjoint aggregate)
    const void *out_grad = nullptr;           // where the last step left dL/dH^(K), and its row pitch
    int out_grad_ld = 0;
};

static thread_local std::string g_create_error;  // errors of calls that have no context: one per host thread

static lp_status fail(lp_ctx *c, lp_status st, const std::string &msg)
{
    if (c) c->err = msg; else g_create_error = msg;
    return st;
}

#define CK(call)                                                                                         \
    do {                                                                                                 \
        cudaError_t e_ = (call);                                                                         \
        if (e_ != cudaSuccess)                                                                           \
            return fail(ctx, e_ == cudaErrorMemoryAllocation ? LP_ENOMEM : LP_ECUDA,                     \
                        std::string(#call) + ": " + cudaGetErrorString(e_));                             \
    } while (0)

#define CK_LAUNCH()                                                                                      \
    do {                                                                                                 \
        cudaError_t e_ = cudaGetLastError();                                                             \
        if (e_ != cudaSuccess) return fail(ctx, LP_ECUDA, std::string("kernel launch: ") + cudaGetErrorString(e_)); \
    } while (0)

template <typename P> static cudaError_t dev_alloc(lp_ctx *c, std::vector<void *> &list, int64_t &bytes_acc, P **out, int64_t count)
{
    size_t bytes = sizeof(P) * (size_t)std::max<int64_t>(count, 1);
    bytes = (bytes + 255) & ~(size_t)255;
    void *p = nullptr;
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { *out = nullptr; return e; }
    list.push_back(p);
    bytes_acc += (int64_t)bytes;
    *out = (P *)p;
    return cudaSuccess;
}
#define GALLOC(ptr, count) CK(dev_alloc(ctx, ctx->graph_allocs, ctx->graph_bytes, &(ptr), (count)))
#define MALLOC(ptr, count) CK(dev_alloc(ctx, ctx->model_allocs, ctx->model_bytes, &(ptr), (count)))

static void free_list(std::vector<void *> &l)
{
    for (void *p : l) cudaFree(p);
    l.clear();
}

// temporaries of one call: released on every way out of it
struct TempAllocs {
    std::vector<void *> list;
    int64_t bytes = 0;
    ~TempAllocs() { free_list(list); }
};

static inline unsigned nblk(int64_t n, int t = 256) { return (unsigned)std::max<int64_t>(1, ceil_div64(n, t)); }

// Algorithmic bytes of one aggregation launch, gather convention: every stored entry reads one
// source row of F elements plus its column index (and coefficient), nothing is assumed cached;
// plus row offsets, the output rows and the optional per-row operands.
template <typename T> static double spmm_bytes(const SpmmArgs<T> &a, int64_t nnz)
{
    const double s = sizeof(T), rows = a.n_rows, F = a.F;
    double b = (double)nnz * (F * s + 4.0 + (a.val ? 4.0 : 0.0)) + (rows + 1.0) * 4.0 + rows * F * s;
    if (a.init) b += rows * F * s;
    if (a.relu_ref) b += rows * F * s;
    if (a.self_out) b += 2.0 * rows * F * s;
    if (a.row_scale) b += rows * 4.0;
    return b;
}
static double gemm_bytes(double M, double N, double K, double s_in, double s_out) { return M * K * s_in + K * N * s_in + M * N * s_out; }

// ----------------------------------------------------------------------------------------------
// load-time kernels
// ----------------------------------------------------------------------------------------------
__global__ void validate_csr_kernel(const int64_t *__restrict__ rowptr64, int n, int64_t nnz, const int *__restrict__ col, int *__restrict__ rowptr32,
                                    int *__restrict__ err)
{
    LP_DEP_ENTER();
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v > n) return;
    const int64_t a = rowptr64[v];
    if (v == 0 && a != 0) atomicOr(err, 1);
    if (v == n) {
        if (a != nnz) atomicOr(err, 2);
        rowptr32[v] = (int)min(max(a, (int64_t)0), nnz);
        return;
    }
    const int64_t b = rowptr64[v + 1];
    if (a < 0 || b < a || b > nnz) { atomicOr(err, 4); rowptr32[v] = (int)min(max(a, (int64_t)0), nnz); return; }
    rowptr32[v] = (int)a;
    int prev = -1;
    for (int64_t e = a; e < b; ++e) {
        const int c = col[e];
        if (c < 0 || c >= n) { atomicOr(err, 8); break; }
        if (c <= prev) { atomicOr(err, 16); break; }
        prev = c;
    }
}

__global__ void degree_kernel(const int *__restrict__ rowptr, const float *__restrict__ w, int n, float *__restrict__ dtilde, float *__restrict__ gcn_self,
                              float *__restrict__ inv_deg)
{
    LP_DEP_ENTER();
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    const int a = rowptr[v], b = rowptr[v + 1];
    float d = 1.f;  // self-loop of weight 1
    if (w) { for (int e = a; e < b; ++e) d += w[e]; } else { d += (float)(b - a); }
    dtilde[v] = d;
    gcn_self[v] = 1.f / d;
    inv_deg[v] = b > a ? 1.f / (float)(b - a) : 0.f;
}

// GCN coefficient of entry e in row v, column u: w_vu / sqrt(d~_v d~_u)
__global__ void gcn_val_kernel(const int *__restrict__ rows, const int *__restrict__ col, const float *__restrict__ w, const float *__restrict__ dtilde,
                               int64_t nnz, float *__restrict__ val)
{
    LP_DEP_ENTER();
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= nnz) return;
    val[e] = (w ? w[e] : 1.f) / sqrtf(dtilde[rows[e]] * dtilde[col[e]]);
}

__global__ void widen_i32_kernel(const int *__restrict__ src, int64_t m, int64_t *__restrict__ dst)
{
    LP_DEP_ENTER();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) dst[i] = src[i];
}

// ----------------------------------------------------------------------------------------------
// life cycle
// ----------------------------------------------------------------------------------------------
extern "C" const char *lp_last_error(const lp_ctx *ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

extern "C" lp_status lp_create(lp_ctx **out, int32_t device, void *cuda_stream)
{
    lp_ctx *ctx = nullptr;
    if (!out) return fail(nullptr, LP_EINVAL, "lp_create: out is NULL");
    *out = nullptr;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess || count <= 0) return fail(nullptr, LP_ECUDA, std::string("lp_create: no CUDA device: ") + cudaGetErrorString(e));
    if (device < 0 || device >= count) return fail(nullptr, LP_EINVAL, "lp_create: device index out of range");
    e = cudaSetDevice(device);
    if (e != cudaSuccess) return fail(nullptr, LP_ECUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(e));
    cudaDeviceProp prop;
    cudaGetDeviceProperties(&prop, device);
    if (prop.major != 10) return fail(nullptr, LP_EUNSUPPORTED, "lp_create: this library is built for sm_100a (B200) only");
    ctx = new (std::nothrow) lp_ctx();
    if (!ctx) return fail(nullptr, LP_ENOMEM, "lp_create: host allocation failed");
    ctx->device = device;
    ctx->ex.st = (cudaStream_t)cuda_stream;
    if (cudaMalloc((void **)&ctx->err_flag, 256) != cudaSuccess || cudaMalloc((void **)&ctx->exhausted_dev, 256) != cudaSuccess ||
        cudaMallocHost((void **)&ctx->host_counts, 64 * sizeof(int)) != cudaSuccess) {
        delete ctx;
        return fail(nullptr, LP_ENOMEM, "lp_create: allocation failed");
    }
    cudaMemset(ctx->err_flag, 0, 256);
    cudaMemset(ctx->exhausted_dev, 0, 256);
    std::string tc_err;
    if (!tc_init(ctx->tc, tc_err)) {
        cudaFree(ctx->err_flag); cudaFree(ctx->exhausted_dev); cudaFreeHost(ctx->host_counts);
        delete ctx;
        return fail(nullptr, LP_ECUDA, "lp_create: " + tc_err);
    }
    *out = ctx;
    return LP_OK;
}

extern "C" void lp_destroy(lp_ctx *ctx)
{
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    cudaStreamSynchronize(ctx->ex.st);
    free_list(ctx->model_allocs);
    free_list(ctx->sparse_allocs);
    free_list(ctx->view_allocs);
    free_list(ctx->graph_allocs);
    tc_destroy(ctx->tc);
    for (cudaEvent_t e : ctx->ex.prof.pool) cudaEventDestroy(e);
    cudaFree(ctx->err_flag);
    cudaFree(ctx->exhausted_dev);
    cudaFreeHost(ctx->host_counts);
    delete ctx;
}

static void drop_model(lp_ctx *ctx)
{
    free_list(ctx->model_allocs);
    ctx->model_bytes = 0;
    ctx->model_set = false;
    ctx->have_forward = ctx->have_grad = false;
    ctx->input_agg_valid = false;
    ctx->hk_valid = false;
    ctx->ex.scan1 = nullptr;
    ctx->scan1 = OnePassScan();
    ctx->w16 = ctx->w16t = ctx->w16s = nullptr;
    for (int l = 0; l < LP_MAX_LAYERS; ++l) { ctx->cat_grad[l] = false; ctx->relu_bits[l] = nullptr; }
    ctx->dcat[0] = ctx->dcat[1] = nullptr;
    ctx->out_grad = nullptr;
    for (auto &l : ctx->layer) l = LayerBuf();
    for (auto &h : ctx->hop) h = HopBlock();
}

// ----------------------------------------------------------------------------------------------
// graph
// ----------------------------------------------------------------------------------------------
extern "C" lp_status lp_load_graph(lp_ctx *ctx, int64_t n, int64_t nnz, const int64_t *rowptr, const int32_t *col, const float *w,
                                   const float *X, int32_t f, int32_t ptrs_on_device)
{
    if (!ctx) return LP_EINVAL;
    if (n <= 0 || n >= (int64_t)1 << 31) return fail(ctx, LP_EINVAL, "lp_load_graph: n must be in [1, 2^31)");
    if (nnz < 0 || nnz >= (int64_t)1 << 31) return fail(ctx, LP_EINVAL, "lp_load_graph: nnz must be in [0, 2^31)");
    if (!rowptr || (!col && nnz > 0) || !X) return fail(ctx, LP_EINVAL, "lp_load_graph: null array");
    if (f <= 0 || f % 8 != 0 || f > 512) return fail(ctx, LP_EINVAL, "lp_load_graph: feature width must be a multiple of 8 in [8, 512]");
    CK(cudaSetDevice(ctx->device));
    CK(cudaStreamSynchronize(ctx->ex.st));
    drop_model(ctx);
    free_list(ctx->sparse_allocs);
    ctx->sp_nnz = -1;
    free_list(ctx->view_allocs);
    ctx->view_nnz = -1;
    free_list(ctx->graph_allocs);
    ctx->graph_bytes = 0;
    ctx->loaded = false;
    ctx->cand = nullptr;
    ctx->n_cand = 0;
    cudaStream_t st = ctx->ex.st;
    const cudaMemcpyKind kind = ptrs_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;

    int64_t *rowptr64 = nullptr;
    TempAllocs tmp_guard;
    std::vector<void *> &tmp = tmp_guard.list;
    int64_t &tmp_bytes = tmp_guard.bytes;
#define TALLOC(ptr, count) CK(dev_alloc(ctx, tmp, tmp_bytes, &(ptr), (count)))
    TALLOC(rowptr64, n + 1);
    GALLOC(ctx->rowptr, n + 1);
    GALLOC(ctx->col, nnz);
    GALLOC(ctx->X32, n * (int64_t)f);
    GALLOC(ctx->X16, n * (int64_t)f);
    if (w) GALLOC(ctx->w, nnz); else ctx->w = nullptr;
    cudaError_t e = cudaMemcpyAsync(rowptr64, rowptr, sizeof(int64_t) * (size_t)(n + 1), kind, st);
    if (e == cudaSuccess && nnz > 0) e = cudaMemcpyAsync(ctx->col, col, sizeof(int) * (size_t)nnz, kind, st);
    if (e == cudaSuccess && w && nnz > 0) e = cudaMemcpyAsync(ctx->w, w, sizeof(float) * (size_t)nnz, kind, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->X32, X, sizeof(float) * (size_t)n * f, kind, st);
    CK(e);

    cudaMemsetAsync(ctx->err_flag, 0, sizeof(int), st);
    launch_dep(validate_csr_kernel, dim3(nblk(n + 1)), dim3(256), 0, st, rowptr64, (int)n, nnz, ctx->col, ctx->rowptr, ctx->err_flag);
    int flag = 0;
    e = cudaMemcpyAsync(&flag, ctx->err_flag, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    CK(e);
    if (flag) {
        free_list(ctx->graph_allocs);
        char buf[160];
        snprintf(buf, sizeof buf, "lp_load_graph: malformed CSR (flags %d: 1/2 rowptr ends, 4 rowptr order, 8 column range, 16 columns not strictly ascending)", flag);
        return fail(ctx, LP_EINVAL, buf);
    }
    ctx->n = (int)n;
    ctx->nnz = nnz;
    ctx->f = f;

    // transposed structure
    GALLOC(ctx->colptr, n + 1);
    GALLOC(ctx->rowidx, nnz);
    GALLOC(ctx->perm, nnz);
    TransposeScratch ts;
    TALLOC(ts.keys, nnz);
    TALLOC(ts.vals, nnz);
    TALLOC(ts.rows, nnz);
    TALLOC(ts.sort.keys_alt, nnz);
    TALLOC(ts.sort.vals_alt, nnz);
    TALLOC(ts.sort.hist, SortScratch::hist_ints(nnz));
    TALLOC(ts.sort.scan_tmp, SortScratch::scan_ints(nnz));
    TALLOC(ts.scan_tmp, ceil_div64(n + 1, SCAN_TILE) + 1);
    transpose_csr(ctx->ex, ctx->rowptr, (int)n, (int)n, ctx->col, nnz, ctx->colptr, ctx->rowidx, ctx->perm, ts);

    // normalisations
    float *dtilde = nullptr;
    TALLOC(dtilde, n);
    GALLOC(ctx->gcn_self, n);
    GALLOC(ctx->inv_deg, n);
    GALLOC(ctx->gcn_val, nnz);
    GALLOC(ctx->gcn_valT, nnz);
    GALLOC(ctx->meanT_val, nnz);
    launch_dep(degree_kernel, dim3(nblk(n)), dim3(256), 0, st, ctx->rowptr, ctx->w, (int)n, dtilde, ctx->gcn_self, ctx->inv_deg);
    if (nnz > 0) {
        launch_dep(gcn_val_kernel, dim3(nblk(nnz)), dim3(256), 0, st, ts.rows, ctx->col, ctx->w, dtilde, nnz, ctx->gcn_val);
        launch_dep(gather_f32_kernel, dim3(nblk(nnz)), dim3(256), 0, st, ctx->gcn_val, ctx->perm, nnz, ctx->gcn_valT);
        launch_dep(gather_f32_kernel, dim3(nblk(nnz)), dim3(256), 0, st, ctx->inv_deg, ctx->rowidx, nnz, ctx->meanT_val);
    }
    launch_dep(convert_kernel<float, bf16>, dim3(nblk(n * (int64_t)f)), dim3(256), 0, st, ctx->X32, ctx->X16, n * (int64_t)f);
    ctx->ex.launches += 6;
    // heavy-row plans of the graph and of its transpose (static: built once)
    const int64_t item_cap = nnz / 64 + 2;  // static plans cut rows above 128 entries into pieces of 128 or items of 512: at most deg / 64 of them per row
    const int static_threshold = 128;  // measured best on a 200k-node power-law graph (64: 282 us, 128: 249 us, 256: 241 us at F=256; 176 / 163 / 193 us at F=128)
    GALLOC(ctx->heavy_partials, item_cap * 512);
    for (HeavyPlan *hp : {&ctx->plan_csr, &ctx->plan_csc}) {
        *hp = HeavyPlan();
        GALLOC(hp->rows, item_cap);
        GALLOC(hp->base, item_cap);
        GALLOC(hp->item_row, item_cap);
        GALLOC(hp->item_first, item_cap);
        GALLOC(hp->nseg, item_cap);
        GALLOC(hp->counts, 64);
        hp->partials = ctx->heavy_partials;
        hp->threshold = static_threshold;
        cudaMemsetAsync(hp->counts, 0, 2 * sizeof(int), st);
        launch_dep(spmm_heavy_plan_kernel, dim3(nblk(n)), dim3(256), 0, st, hp == &ctx->plan_csr ? ctx->rowptr : ctx->colptr, (int)n, nullptr, *hp, nullptr);
        cudaMemcpyAsync(ctx->host_counts + (hp == &ctx->plan_csr ? 0 : 2), hp->counts, 2 * sizeof(int), cudaMemcpyDeviceToHost, st);
    }
    ctx->ex.launches += 2;
    e = cudaStreamSynchronize(st);
    // padded form of both structures (for spmm_padded_kernel), with the GCN coefficients padded alongside
    static_assert(SPMM_PIECE % 4 == 0, "pieces are whole groups");
    for (HeavyPlan *hp : {&ctx->plan_csr, &ctx->plan_csc}) {
        if (e != cudaSuccess || n <= 0 || n >= (1 << 27) || item_cap >= (1 << 27)) break;  // row and slot numbers share 27 bits of the finishing codes
        const bool csr = hp == &ctx->plan_csr;
        const int *sp = csr ? ctx->rowptr : ctx->colptr, *sc = csr ? ctx->col : ctx->rowidx;
        const float *sv = csr ? ctx->gcn_val : ctx->gcn_valT;
        // heavy rows of the padded form: pieces of SPMM_PIECE entries, one partial slot each
        HeavyPlan pp;
        GALLOC(pp.rows, item_cap);
        GALLOC(pp.base, item_cap);
        GALLOC(pp.nseg, item_cap);
        GALLOC(pp.counts, 64);
        TALLOC(pp.item_row, item_cap);
        TALLOC(pp.item_first, item_cap);
        pp.threshold = SPMM_PIECE;
        pp.seg = SPMM_PIECE;
        int *row_base = nullptr, *first_group = nullptr, *chunk_count = nullptr, *chunk_of = nullptr;
        TALLOC(row_base, n + 1);
        TALLOC(first_group, n + 1);
        TALLOC(chunk_count, n + 1);
        TALLOC(chunk_of, n + 1);
        cudaMemsetAsync(pp.counts, 0, 2 * sizeof(int), st);
        launch_dep(spmm_heavy_plan_kernel, dim3(nblk(n)), dim3(256), 0, st, sp, (int)n, nullptr, pp, row_base);
        launch_dep(padded_count_kernel, dim3(nblk(n)), dim3(256), 0, st, sp, (int)n, SPMM_PIECE, first_group);
        exclusive_scan_i32(ctx->ex, first_group, n, first_group, first_group + n, ts.scan_tmp);
        launch_dep(padded_chunk_count_kernel, dim3(nblk(n)), dim3(256), 0, st, sp, first_group, (int)n, SPMM_PIECE, chunk_count);
        exclusive_scan_i32(ctx->ex, chunk_count, n, chunk_of, chunk_of + n, ts.scan_tmp);
        cudaMemcpyAsync(ctx->host_counts + 8, first_group + n, sizeof(int), cudaMemcpyDeviceToHost, st);
        cudaMemcpyAsync(ctx->host_counts + 9, chunk_of + n, sizeof(int), cudaMemcpyDeviceToHost, st);
        cudaMemcpyAsync(ctx->host_counts + 10, pp.counts, 2 * sizeof(int), cudaMemcpyDeviceToHost, st);
        e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) break;
        const int64_t n_groups = ctx->host_counts[8];
        const int n_chunks = ctx->host_counts[9];
        if (ctx->host_counts[11] > item_cap) break;  // cannot happen (a piece has at least 1 entry of a row with more than 128): keep the row-per-group kernel
        int *pcol = nullptr, *grow = nullptr, *chunk_start = nullptr;
        float *pval = nullptr;
        GALLOC(pcol, 4 * n_groups + 4);
        GALLOC(pval, 4 * n_groups + 4);
        GALLOC(grow, n_groups + 1);
        GALLOC(chunk_start, (int64_t)n_chunks + 2);
        launch_dep(padded_fill_kernel, dim3(nblk(n)), dim3(256), 0, st, sp, sc, sv, (int)n, SPMM_PIECE, first_group, chunk_count, chunk_of, row_base, chunk_start, pcol, pval, grow);
        ctx->ex.launches += 5;
        e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) break;
        hp->pcol = reinterpret_cast<const int4 *>(pcol);
        hp->pval = reinterpret_cast<const float4 *>(pval);
        hp->pval_src = sv;
        if (!csr) {  // the transposed structure also carries the mean's coefficients 1 / |N(v)| of the entry's source row v
            float *pval2 = nullptr;
            GALLOC(pval2, 4 * n_groups + 4);
            launch_dep(padded_fill_kernel, dim3(nblk(n)), dim3(256), 0, st, sp, sc, ctx->meanT_val, (int)n, SPMM_PIECE, first_group, chunk_count, chunk_of, row_base, chunk_start, pcol, pval2, grow);
            ctx->ex.launches += 1;
            e = cudaStreamSynchronize(st);
            if (e != cudaSuccess) break;
            hp->pval2 = reinterpret_cast<const float4 *>(pval2);
            hp->pval2_src = ctx->meanT_val;
        }
        hp->grow = grow;
        hp->chunk_start = chunk_start;
        hp->n_chunks = n_groups > 0 ? n_chunks : 0;
        hp->p_rows = pp.rows;
        hp->p_base = pp.base;
        hp->p_counts = pp.counts;
        hp->p_nseg = pp.nseg;
        hp->p_host_rows = ctx->host_counts[10];
    }
#undef TALLOC
    CK(e);
    CK_LAUNCH();
    ctx->plan_csr.host_rows = ctx->host_counts[0];
    ctx->plan_csr.host_items = ctx->host_counts[1];
    ctx->plan_csc.host_rows = ctx->host_counts[2];
    ctx->plan_csc.host_items = ctx->host_counts[3];
    ctx->plan_dyn = HeavyPlan();
    ctx->loaded = true;
    return LP_OK;
}

extern "C" lp_status lp_get_structure(lp_ctx *ctx, int64_t *colptr, int32_t *rowidx, int64_t *perm)
{
    if (!ctx) return LP_EINVAL;
    if (!ctx->loaded) return fail(ctx, LP_ESTATE, "lp_get_structure: no graph loaded");
    CK(cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->ex.st;
    if (colptr) launch_dep(widen_i32_kernel, dim3(nblk(ctx->n + 1)), dim3(256), 0, st, ctx->colptr, ctx->n + 1, colptr);
    if (rowidx && ctx->nnz > 0) CK(cudaMemcpyAsync(rowidx, ctx->rowidx, sizeof(int) * (size_t)ctx->nnz, cudaMemcpyDeviceToDevice, st));
    if (perm && ctx->nnz > 0) launch_dep(widen_i32_kernel, dim3(nblk(ctx->nnz)), dim3(256), 0, st, ctx->perm, ctx->nnz, perm);
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_set_candidates(lp_ctx *ctx, const int32_t *cand, int64_t n_cand)
{
    if (!ctx) return LP_EINVAL;
    if (!ctx->loaded) return fail(ctx, LP_ESTATE, "lp_set_candidates: no graph loaded");
    CK(cudaSetDevice(ctx->device));
    CK(cudaStreamSynchronize(ctx->ex.st));  // earlier sampling launches may still read the previous set
    if (ctx->cand) {                        // the previous set is released: repeated calls do not grow the context
        auto it = std::find(ctx->graph_allocs.begin(), ctx->graph_allocs.end(), (void *)ctx->cand);
        if (it != ctx->graph_allocs.end()) ctx->graph_allocs.erase(it);
        cudaFree(ctx->cand);
        ctx->cand = nullptr;
        ctx->n_cand = 0;
    }
    if (!cand || n_cand <= 0) return LP_OK;
    if (n_cand >= (int64_t)1 << 31) return fail(ctx, LP_EINVAL, "lp_set_candidates: too many candidates");
    GALLOC(ctx->cand, n_cand);  // lives with the graph
    CK(cudaMemcpyAsync(ctx->cand, cand, sizeof(int) * (size_t)n_cand, cudaMemcpyDeviceToDevice, ctx->ex.st));
    launch_dep(check_ids_kernel, dim3(nblk(n_cand)), dim3(256), 0, ctx->ex.st, ctx->cand, n_cand, ctx->n, ctx->err_flag);
    int bad = 0;
    CK(cudaMemcpyAsync(&bad, ctx->err_flag, sizeof bad, cudaMemcpyDeviceToHost, ctx->ex.st));
    CK(cudaStreamSynchronize(ctx->ex.st));
    if (bad) {
        cudaMemsetAsync(ctx->err_flag, 0, sizeof(int), ctx->ex.st);
        ctx->graph_allocs.erase(std::find(ctx->graph_allocs.begin(), ctx->graph_allocs.end(), (void *)ctx->cand));
        cudaFree(ctx->cand);
        ctx->cand = nullptr;
        return fail(ctx, LP_EINVAL, "lp_set_candidates: candidate id outside [0, n)");
    }
    ctx->n_cand = n_cand;
    return LP_OK;
}

// ----------------------------------------------------------------------------------------------
// sparsification
// ----------------------------------------------------------------------------------------------
static lp_status sync_counts(lp_ctx *ctx, const int *dev_a, const int *dev_b, int *out_a, int *out_b);

#define SALLOC(ptr, count) CK(dev_alloc(ctx, ctx->sparse_allocs, ctx->sparse_bytes, &(ptr), (count)))

extern "C" lp_status lp_sparsify(lp_ctx *ctx, double alpha, uint64_t seed, int64_t *nnz_out)
{
    if (!ctx || !nnz_out) return LP_EINVAL;
    if (!ctx->loaded) return fail(ctx, LP_ESTATE, "lp_sparsify: no graph loaded");
    if (!(alpha > 0.0) || alpha > 1e6) return fail(ctx, LP_EINVAL, "lp_sparsify: alpha must be in (0, 1e6]");
    CK(cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->ex.st;
    CK(cudaStreamSynchronize(st));
    free_list(ctx->sparse_allocs);
    ctx->sparse_bytes = 0;
    ctx->sp_nnz = -1;
    const int n = ctx->n;
    const int64_t nnz = ctx->nnz;
    const int64_t L = (int64_t)std::floor(alpha * (double)(nnz / 2));
    int *flags = nullptr, *pos = nullptr, *nz = nullptr, *hits = nullptr, *scan_tmp = nullptr;
    const int64_t m = std::max<int64_t>(n, nnz) + 2;
    SALLOC(flags, m);
    SALLOC(pos, m);
    SALLOC(nz, n + 1);
    SALLOC(hits, nnz + 1);
    SALLOC(scan_tmp, ceil_div64(m, SCAN_TILE) + 2);
    SALLOC(ctx->sp_ptr, n + 1);
    // non-isolated nodes, ascending
    launch_dep(sp_nonisolated_kernel, dim3(nblk(n)), dim3(256), 0, st, ctx->rowptr, n, flags);
    exclusive_scan_i32(ctx->ex, flags, n, pos, pos + n, scan_tmp);
    launch_dep(sp_compact_kernel, dim3(nblk(n)), dim3(256), 0, st, ctx->rowptr, pos, n, nz);
    int n_nz = 0, dummy = 0;
    lp_status s = sync_counts(ctx, pos + n, nullptr, &n_nz, &dummy);
    if (s != LP_OK) return s;
    CK(cudaMemsetAsync(hits, 0, sizeof(int) * (size_t)(nnz + 1), st));
    CK(cudaMemsetAsync(ctx->err_flag, 0, sizeof(int), st));
    if (L > 0 && n_nz > 0)
        launch_dep(sp_draw_kernel, dim3(nblk(L)), dim3(256), 0, st, ctx->rowptr, ctx->col, nz, (uint32_t)n_nz, make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)), L, hits,
                                                ctx->err_flag);
    // kept entries -> positions; pos has nnz + 1 slots so that pos[rowptr[n]] is the total
    launch_dep(sp_keep_flags_kernel, dim3(nblk(nnz + 1)), dim3(256), 0, st, hits, nnz + 1, flags);
    exclusive_scan_i32(ctx->ex, flags, nnz + 1, pos, nullptr, scan_tmp);
    int kept = 0, bad = 0;
    s = sync_counts(ctx, pos + nnz, ctx->err_flag, &kept, &bad);
    if (s != LP_OK) return s;
    if (bad) {
        cudaMemsetAsync(ctx->err_flag, 0, sizeof(int), st);
        return fail(ctx, LP_EINVAL, "lp_sparsify: the loaded graph is not symmetric (a drawn entry has no mirror)");
    }
    SALLOC(ctx->sp_col, kept);
    SALLOC(ctx->sp_w, kept);
    launch_dep(sp_emit_kernel, dim3(nblk(n + 1)), dim3(256), 0, st, ctx->rowptr, ctx->col, hits, pos, n, (double)n_nz, (double)std::max<int64_t>(L, 1), ctx->sp_ptr, ctx->sp_col,
                                                ctx->sp_w);
    ctx->ex.launches += 5;
    CK(cudaStreamSynchronize(st));
    CK_LAUNCH();
    ctx->sp_nnz = kept;
    *nnz_out = kept;
    return LP_OK;
}

extern "C" lp_status lp_get_sparsified(lp_ctx *ctx, int64_t *rowptr, int32_t *col, float *w)
{
    if (!ctx) return LP_EINVAL;
    if (ctx->sp_nnz < 0) return fail(ctx, LP_ESTATE, "lp_get_sparsified: call lp_sparsify first");
    CK(cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->ex.st;
    if (rowptr) CK(cudaMemcpyAsync(rowptr, ctx->sp_ptr, sizeof(int64_t) * ((size_t)ctx->n + 1), cudaMemcpyDeviceToDevice, st));
    if (col && ctx->sp_nnz > 0) CK(cudaMemcpyAsync(col, ctx->sp_col, sizeof(int) * (size_t)ctx->sp_nnz, cudaMemcpyDeviceToDevice, st));
    if (w && ctx->sp_nnz > 0) CK(cudaMemcpyAsync(w, ctx->sp_w, sizeof(float) * (size_t)ctx->sp_nnz, cudaMemcpyDeviceToDevice, st));
    return LP_OK;
}

// ----------------------------------------------------------------------------------------------
// worker view
// ----------------------------------------------------------------------------------------------
#define VALLOC(ptr, count) CK(dev_alloc(ctx, ctx->view_allocs, ctx->view_bytes, &(ptr), (count)))

extern "C" lp_status lp_worker_view(lp_ctx *ctx, const int32_t *part, int32_t worker, int32_t keep_cross_edges, int32_t foreign_mode,
                                    int64_t *nnz_out, lp_view_stats *stats)
{
    if (!ctx || !nnz_out) return LP_EINVAL;
    if (!ctx->loaded) return fail(ctx, LP_ESTATE, "lp_worker_view: no graph loaded");
    if (!part) return fail(ctx, LP_EINVAL, "lp_worker_view: part is NULL");
    if (foreign_mode < 0 || foreign_mode > 2) return fail(ctx, LP_EINVAL, "lp_worker_view: foreign_mode must be 0, 1 or 2");
    if (foreign_mode == VIEW_FOREIGN_SPARSIFIED && ctx->sp_nnz < 0) return fail(ctx, LP_ESTATE, "lp_worker_view: call lp_sparsify first");
    CK(cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->ex.st;
    CK(cudaStreamSynchronize(st));
    free_list(ctx->view_allocs);
    ctx->view_bytes = 0;
    ctx->view_nnz = -1;
    const int n = ctx->n;
    int *scan_tmp = nullptr;
    unsigned long long *dstats = nullptr;
    VALLOC(ctx->view_ptr, n + 1);
    VALLOC(scan_tmp, ceil_div64(n + 1, SCAN_TILE) + 2);
    VALLOC(dstats, 8);
    CK(cudaMemsetAsync(dstats, 0, 8 * sizeof(unsigned long long), st));
    launch_dep(view_count_kernel, dim3(nblk(n)), dim3(256), 0, st, n, ctx->rowptr, ctx->col, part, worker, keep_cross_edges, foreign_mode, ctx->sp_ptr, ctx->view_ptr, dstats);
    exclusive_scan_i32(ctx->ex, ctx->view_ptr, n, ctx->view_ptr, ctx->view_ptr + n, scan_tmp);
    unsigned long long hs[4] = {0, 0, 0, 0};
    CK(cudaMemcpyAsync(hs, dstats, sizeof hs, cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    const unsigned long long total = hs[0] + hs[1];
    if (total >= (1ull << 31)) return fail(ctx, LP_EINVAL, "lp_worker_view: the view has 2^31 entries or more");
    VALLOC(ctx->view_col, (int64_t)total);
    launch_dep(view_fill_kernel, dim3(nblk(n)), dim3(256), 0, st, n, ctx->rowptr, ctx->col, part, worker, keep_cross_edges, foreign_mode, ctx->sp_ptr, ctx->sp_col,
                                              ctx->view_ptr, ctx->view_col);
    ctx->ex.launches += 2;
    CK(cudaStreamSynchronize(st));
    CK_LAUNCH();
    ctx->view_nnz = (int64_t)total;
    *nnz_out = (int64_t)total;
    if (stats) {
        stats->own_entries = (int64_t)hs[0];
        stats->foreign_entries = (int64_t)hs[1];
        stats->foreign_rows = (int64_t)hs[2];
        stats->own_nodes = (int64_t)hs[3];
    }
    return LP_OK;
}

extern "C" lp_status lp_get_worker_view(lp_ctx *ctx, int64_t *rowptr, int32_t *col)
{
    if (!ctx) return LP_EINVAL;
    if (ctx->view_nnz < 0) return fail(ctx, LP_ESTATE, "lp_get_worker_view: call lp_worker_view first");
    CK(cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->ex.st;
    if (rowptr) launch_dep(widen_i32_kernel, dim3(nblk(ctx->n + 1)), dim3(256), 0, st, ctx->view_ptr, ctx->n + 1, rowptr);
    if (col && ctx->view_nnz > 0) CK(cudaMemcpyAsync(col, ctx->view_col, sizeof(int) * (size_t)ctx->view_nnz, cudaMemcpyDeviceToDevice, st));
    CK_LAUNCH();
    return LP_OK;
}

// ----------------------------------------------------------------------------------------------
// model
// ----------------------------------------------------------------------------------------------
extern "C" lp_status lp_param_count(const lp_ctx *ctx, int64_t *n_params)
{
    if (!ctx || !n_params) return LP_EINVAL;
    if (!ctx->model_set) return fail(const_cast<lp_ctx *>(ctx), LP_ESTATE, "lp_param_count: no model set");
    *n_params = ctx->n_params;
    return LP_OK;
}

extern "C" lp_status lp_set_model(lp_ctx *ctx, const lp_model_desc *d, int64_t max_batch, int32_t max_k)
{
    if (!ctx || !d) return LP_EINVAL;
    if (!ctx->loaded) return fail(ctx, LP_ESTATE, "lp_set_model: load a graph first");
    if (d->arch != LP_GCN && d->arch != LP_SAGE_MEAN) return fail(ctx, LP_EINVAL, "lp_set_model: unknown architecture");
    if (d->prec != LP_FP32 && d->prec != LP_BF16) return fail(ctx, LP_EINVAL, "lp_set_model: unknown precision");
    if (d->n_layers < 1 || d->n_layers > LP_MAX_LAYERS) return fail(ctx, LP_EINVAL, "lp_set_model: n_layers out of range");
    if (d->dims[0] != ctx->f) return fail(ctx, LP_EINVAL, "lp_set_model: dims[0] differs from the feature width of the graph");
    const int align = d->prec == LP_BF16 ? 64 : 8;
    for (int k = 0; k <= d->n_layers; ++k)
        if (d->dims[k] <= 0 || d->dims[k] % align != 0 || d->dims[k] > 512)
            return fail(ctx, LP_EINVAL, "lp_set_model: widths must be multiples of 8 (FP32) or 64 (BF16), at most 512");
    bool sampled = false;
    for (int h = 0; h < d->n_layers; ++h) {
        if (d->fanout[h] < 0 || d->fanout[h] > MAX_FANOUT) return fail(ctx, LP_EINVAL, "lp_set_model: fanout must be in [0, 32]");
        sampled |= d->fanout[h] > 0;
    }
    if (sampled) {
        for (int h = 0; h < d->n_layers; ++h)
            if (d->fanout[h] == 0) return fail(ctx, LP_EINVAL, "lp_set_model: fanouts must be all zero or all positive");
        if (d->cache_input_aggregation) return fail(ctx, LP_EINVAL, "lp_set_model: cache_input_aggregation needs a full-graph model (sampled neighbourhoods change every step)");
    }
    if (d->predictor != LP_PRED_DOT && d->predictor != LP_PRED_MLP) return fail(ctx, LP_EINVAL, "lp_set_model: unknown predictor");
    if (d->predictor == LP_PRED_MLP && (d->pred_hidden <= 0 || d->pred_hidden % align != 0 || d->pred_hidden > 512))
        return fail(ctx, LP_EINVAL, "lp_set_model: pred_hidden must be a multiple of 8 (FP32) or 64 (BF16), at most 512");
    if (max_batch <= 0 || max_k < 0 || max_k > 255) return fail(ctx, LP_EINVAL, "lp_set_model: max_batch must be positive, max_k in [0, 255]");
    if (d->reject_edges && (d->max_attempts < 1 || d->max_attempts > 255)) return fail(ctx, LP_EINVAL, "lp_set_model: max_attempts must be in [1, 255]");
    if (max_batch * (int64_t)(1 + max_k) * 2 >= (int64_t)1 << 31) return fail(ctx, LP_EINVAL, "lp_set_model: batch too large");
    CK(cudaSetDevice(ctx->device));
    CK(cudaStreamSynchronize(ctx->ex.st));
    drop_model(ctx);
    ctx->desc = *d;
    ctx->K = d->n_layers;
    ctx->sampled = sampled;
    ctx->max_batch = max_batch;
    ctx->max_k = max_k;
    const int K = ctx->K;
    const size_t es = d->prec == LP_BF16 ? 2 : 4;
    const bool sage = d->arch == LP_SAGE_MEAN;
    const int64_t n = ctx->n;
    const int64_t E = max_batch * (1 + (int64_t)max_k);

    int64_t off = 0;
    for (int k = 0; k < K; ++k) {
        LayerBuf &L = ctx->layer[k];
        L.Fi = d->dims[k];
        L.Fo = d->dims[k + 1];
        L.Kin = sage ? 2 * L.Fi : L.Fi;
        L.off_w = off;
        off += (int64_t)L.Kin * L.Fo;
        L.off_b = off;
        off += L.Fo;
    }
    ctx->n_enc_params = off;
    ctx->mlp = d->predictor == LP_PRED_MLP;
    ctx->Hp = ctx->mlp ? d->pred_hidden : 0;
    if (ctx->mlp) {
        const int Dk = d->dims[K], Hp = ctx->Hp;
        LayerBuf &P0 = ctx->pred[0], &P1 = ctx->pred[1];
        P0 = LayerBuf(); P1 = LayerBuf();
        P0.Fi = P0.Kin = Dk; P0.Fo = Hp; P0.off_w = off; off += (int64_t)Dk * Hp; P0.off_b = off; off += Hp;
        P1.Fi = P1.Kin = Hp; P1.Fo = Hp; P1.off_w = off; off += (int64_t)Hp * Hp; P1.off_b = off; off += Hp;
        ctx->off_w2 = off; off += Hp;
        ctx->off_b2 = off; off += 1;
    }
    ctx->n_params = off;

    // row capacities per hop (frontier sizes are bounded by n and by the fan-out product)
    int64_t cap_rows[LP_MAX_LAYERS + 1];
    if (sampled) {
        cap_rows[0] = std::min<int64_t>(n, max_batch * (2 + 2 * (int64_t)max_k));
        for (int h = 1; h <= K; ++h) cap_rows[h] = std::min<int64_t>(n, cap_rows[h - 1] * (1 + (int64_t)d->fanout[h - 1]));
    } else {
        for (int h = 0; h <= K; ++h) cap_rows[h] = n;
    }
    int64_t max_rows = 0;
    for (int h = 0; h <= K; ++h) max_rows = std::max(max_rows, cap_rows[h]);
    int maxF = 0, maxKin = 0;
    for (int k = 0; k < K; ++k) { maxF = std::max(maxF, std::max(ctx->layer[k].Fi, ctx->layer[k].Fo)); maxKin = std::max(maxKin, ctx->layer[k].Kin); }

    char *p = nullptr;
    for (int k = 0; k < K; ++k) {
        LayerBuf &L = ctx->layer[k];
        // rows of layer k: destinations of hop K-k  (F_{K-k-1}); full graph: n
        const int64_t rows = sampled ? cap_rows[K - k - 1] : n;
        MALLOC(p, rows * L.Kin * (int64_t)es);
        L.A = p;
        if (!sage && !sampled) {
            if (k == 0) {
                L.Hin = d->prec == LP_BF16 ? (void *)ctx->X16 : (void *)ctx->X32;
            } else {
                MALLOC(p, n * L.Fi * (int64_t)es);
                L.Hin = p;
            }
        }
        if (sampled && k < K - 1) {
            MALLOC(p, rows * L.Fo * (int64_t)es);
            L.Hout = p;
        }
    }
    {
        const int64_t rows = sampled ? cap_rows[0] : n;
        MALLOC(p, rows * d->dims[K] * (int64_t)es);
        ctx->HK = p;
        MALLOC(p, rows * d->dims[K] * (int64_t)es);
        ctx->dHK = p;
    }
    if (sage && !sampled) {  // the left half of the first operand is X itself, written once
        LayerBuf &L = ctx->layer[0];
        if (d->prec == LP_BF16)
            launch_dep(copy_rows_kernel<bf16, bf16>, dim3(nblk(n * L.Fi)), dim3(256), 0, ctx->ex.st, ctx->X16, L.Fi, (bf16 *)L.A, L.Kin, n, L.Fi);
        else
            launch_dep(copy_rows_kernel<float, float>, dim3(nblk(n * L.Fi)), dim3(256), 0, ctx->ex.st, ctx->X32, L.Fi, (float *)L.A, L.Kin, n, L.Fi);
        ctx->ex.launches += 1;
    }
    for (int i = 0; i < 2; ++i) { MALLOC(p, max_rows * maxF * (int64_t)es); ctx->dZ[i] = p; }
    MALLOC(p, max_rows * maxKin * (int64_t)es);
    ctx->dA = p;
    int64_t part_rows = max_rows;
    if (ctx->mlp) {  // the predictor's layers run over the scored edges
        part_rows = std::max<int64_t>(part_rows, E);
        maxKin = std::max(maxKin, std::max(d->dims[K], ctx->Hp));
        maxF = std::max(maxF, std::max(d->dims[K], ctx->Hp));
    }
    ctx->partials_floats = std::max<int64_t>((int64_t)weight_grad_splits(part_rows) * maxKin * maxF, (int64_t)colsum_splits(part_rows) * (maxF + 1));
    ctx->partials_floats = std::max<int64_t>(ctx->partials_floats, tc_weight_grad_partials(part_rows, maxKin, maxF));
    MALLOC(ctx->partials, ctx->partials_floats);

    // scoring and incidence
    MALLOC(ctx->g_pos, ctx->mlp ? E : max_batch);  // MLP predictor: one array for positives then negatives
    MALLOC(ctx->g_neg, max_batch * std::max<int64_t>(max_k, 1));
    MALLOC(ctx->loss_partials, std::max<int64_t>(ceil_div64(max_batch, EDGE_THREADS / 32), ceil_div64(E, 256)) + 1);
    if (ctx->mlp) {
        const int Dk = d->dims[K], Hp = ctx->Hp;
        MALLOC(p, E * Dk * (int64_t)es); ctx->pred[0].A = p;
        MALLOC(p, E * Hp * (int64_t)es); ctx->pred[1].A = p;
        MALLOC(p, E * Hp * (int64_t)es); ctx->P2 = p;
        MALLOC(p, E * Hp * (int64_t)es); ctx->dPa = p;
        MALLOC(p, E * Hp * (int64_t)es); ctx->dPb = p;
        MALLOC(p, E * Dk * (int64_t)es); ctx->dZ0 = p;
        MALLOC(ctx->pred_scores, E);
        MALLOC(ctx->inc_edge, 2 * E);
    }
    MALLOC(ctx->inc_cursor, cap_rows[0] + 1);
    MALLOC(ctx->inc_partials, (2 * E / SPMM_HEAVY_MIN + 2) * 2 * (int64_t)d->dims[K]);
    MALLOC(ctx->inc_col, 2 * E);
    MALLOC(ctx->inc_val, 2 * E);
    MALLOC(ctx->inc_ptr, cap_rows[0] + 1);
    ctx->inc_cap = cap_rows[0] + 1;
    MALLOC(ctx->d_pos_tmp, 2 * max_batch);
    MALLOC(ctx->d_neg_tmp, max_batch * std::max<int64_t>(max_k, 1));
    MALLOC(ctx->d_loss_tmp, 64);
    MALLOC(ctx->d_grads_tmp, ctx->n_params);
    if (d->prec == LP_BF16) {
        MALLOC(ctx->w16, ctx->n_params);
        MALLOC(ctx->w16t, ctx->n_params);
        // layers whose input gradient is taken as aggregate-then-transform (see cat_grad): the widths must suit the pair
        // kernel in both directions and the padded adjoint, and aggregating dZ (Fo wide) must not cost more than
        // aggregating the transformed gradient (Fi wide)
        int max_fo = 0;
        for (int l = 1; l < K && sage && !sampled; ++l) {
            const LayerBuf &L = ctx->layer[l], &P = ctx->layer[l - 1];
            if (L.Fo <= L.Fi && L.Fi % 32 == 0 && ctx->plan_csc.pval2 && tc_linear_supported(2 * L.Fo, L.Fi) && tc_pair_applies(n, L.Fi, 2 * L.Fo) &&
                tc_linear_supported(P.Kin, P.Fo) && tc_pair_applies(n, P.Fo, P.Kin)) {
                ctx->cat_grad[l] = true;
                MALLOC(ctx->relu_bits[l], (int64_t)(L.Fi / 32) * n);
                max_fo = std::max(max_fo, L.Fo);
            }
        }
        if (max_fo > 0) {
            MALLOC(ctx->w16s, ctx->n_params);
            for (int i = 0; i < 2; ++i) { MALLOC(p, n * 2 * (int64_t)max_fo * es); ctx->dcat[i] = p; }
        }
    }

    // per-step sort capacity: incidence lists and (sampled) block transposes
    int64_t sort_cap = 2 * E;
    if (sampled) {
        for (int h = 1; h <= K; ++h) {
            HopBlock &hb = ctx->hop[h];
            hb.cap_dst = (int)cap_rows[h - 1];
            hb.cap_src = (int)cap_rows[h];
            hb.cap_entries = (int64_t)hb.cap_dst * d->fanout[h - 1];
            if (hb.cap_entries >= (int64_t)1 << 31) return fail(ctx, LP_EINVAL, "lp_set_model: sampled block too large");
            if (h < K) sort_cap = std::max(sort_cap, hb.cap_entries);
        }
        ctx->hop[0].cap_src = (int)cap_rows[0];
        for (int h = 0; h <= K; ++h) {
            HopBlock &hb = ctx->hop[h];
            MALLOC(hb.n_front_dev, 64);
            if (h < K) {  // the outermost frontier is never materialised: layer 1 reads X by global id
                MALLOC(hb.frontier, hb.cap_src);
                MALLOC(hb.posmap, n);
            }
            if (h >= 1) {
                MALLOC(hb.blk_ptr, (int64_t)hb.cap_dst + 1);
                MALLOC(hb.blk_col_global, hb.cap_entries);
                MALLOC(hb.blk_row, hb.cap_entries);
                MALLOC(hb.inv_deg, hb.cap_dst);
                if (!sage) {
                    MALLOC(hb.blk_eid, hb.cap_entries);
                    MALLOC(hb.blk_val, hb.cap_entries);
                    MALLOC(hb.self_coef_dst, hb.cap_dst);
                    if (h < K) {
                        MALLOC(hb.blk_valT, hb.cap_entries);
                        MALLOC(hb.self_coef_src, hb.cap_src);
                    }
                }
                if (h < K) {
                    MALLOC(hb.blk_col_local, hb.cap_entries);
                    MALLOC(hb.colptr, (int64_t)hb.cap_src + 1);
                    MALLOC(hb.rowidx, hb.cap_entries);
                    MALLOC(hb.perm, hb.cap_entries);
                    MALLOC(hb.self_idx, hb.cap_dst);
                    MALLOC(hb.inv_self, hb.cap_src);
                }
            }
        }
        MALLOC(ctx->mark, n);
        MALLOC(ctx->flags, n);
        MALLOC(ctx->seed_ids, max_batch * (2 + 2 * (int64_t)max_k));
    }
    {   // heavy-row plan scratch for the per-step structures (incidence lists, sampled blocks)
        int64_t dyn_nnz = 2 * E;
        if (sampled)
            for (int h = 1; h <= K; ++h) dyn_nnz = std::max(dyn_nnz, ctx->hop[h].cap_entries);
        const int64_t cap = dyn_nnz / SPMM_HEAVY_MIN + 2;
        HeavyPlan &hp = ctx->plan_dyn;
        hp = HeavyPlan();
        MALLOC(hp.rows, cap);
        MALLOC(hp.base, cap);
        MALLOC(hp.item_row, cap);
        MALLOC(hp.item_first, cap);
        MALLOC(hp.nseg, cap);
        MALLOC(hp.counts, 64);
        if (cap > ctx->nnz / 64 + 2) {  // larger than the partial rows allocated with the graph
            MALLOC(hp.partials, cap * 512);
        } else {
            hp.partials = ctx->heavy_partials;
        }
    }
    ctx->sort_cap = sort_cap;
    MALLOC(ctx->sort.keys_alt, sort_cap);
    MALLOC(ctx->sort.vals_alt, sort_cap);
    MALLOC(ctx->sort.hist, SortScratch::hist_ints(sort_cap));
    MALLOC(ctx->sort.scan_tmp, SortScratch::scan_ints(sort_cap));
    MALLOC(ctx->tsp.keys, sort_cap);
    MALLOC(ctx->tsp.vals, sort_cap);
    MALLOC(ctx->tsp.rows, sort_cap);
    ctx->tsp.sort = ctx->sort;
    MALLOC(ctx->scan_tmp, ceil_div64(n + 1, SCAN_TILE) + 2);
    ctx->tsp.scan_tmp = ctx->scan_tmp;
    ctx->scan1 = OnePassScan();
    ctx->scan1.tiles_cap = std::max<int64_t>(ceil_div64(n + 1, SCAN_TILE), ceil_div64(SortScratch::hist_ints(sort_cap), SCAN_TILE)) + 1;
    MALLOC(ctx->scan1.status, ctx->scan1.tiles_cap);
    MALLOC(ctx->scan1.ticket, 64);
    CK(cudaMemsetAsync(ctx->scan1.status, 0, sizeof(unsigned long long) * (size_t)ctx->scan1.tiles_cap, ctx->ex.st));
    CK(cudaMemsetAsync(ctx->scan1.ticket, 0, 64 * sizeof(unsigned), ctx->ex.st));
    ctx->ex.scan1 = &ctx->scan1;  // from here on every scan of this context takes one launch
    ctx->ex.scan_err = ctx->err_flag;
    CK(cudaStreamSynchronize(ctx->ex.st));
    CK_LAUNCH();
    ctx->model_set = true;
    return LP_OK;
}

// ----------------------------------------------------------------------------------------------
// negatives
// ----------------------------------------------------------------------------------------------
extern "C" lp_status lp_sample_negatives(lp_ctx *ctx, uint64_t seed, uint64_t step, int32_t k, int32_t mode, const int32_t *pos_src,
                                         int64_t B, int64_t edge_index_base, int32_t *neg_src, int32_t *neg_dst)
{
    if (!ctx) return LP_EINVAL;
    if (!ctx->loaded) return fail(ctx, LP_ESTATE, "lp_sample_negatives: no graph loaded");
    if (k < 0 || k > 255 || B < 0 || edge_index_base < 0) return fail(ctx, LP_EINVAL, "lp_sample_negatives: k in [0, 255], B >= 0, base >= 0");
    if (mode != LP_NEG_PER_SOURCE && mode != LP_NEG_GLOBAL_PAIR) return fail(ctx, LP_EINVAL, "lp_sample_negatives: unknown mode");
    if (B * (int64_t)k == 0) return LP_OK;
    if (!neg_dst) return fail(ctx, LP_EINVAL, "lp_sample_negatives: neg_dst is NULL");
    if (mode == LP_NEG_PER_SOURCE && !pos_src) return fail(ctx, LP_EINVAL, "lp_sample_negatives: pos_src is NULL");
    if (mode == LP_NEG_GLOBAL_PAIR && !neg_src) return fail(ctx, LP_EINVAL, "lp_sample_negatives: global-pair mode needs neg_src");
    CK(cudaSetDevice(ctx->device));
    const int reject = ctx->model_set ? ctx->desc.reject_edges : 1;
    const int attempts = (ctx->model_set && ctx->desc.reject_edges) ? ctx->desc.max_attempts : (reject ? 8 : 1);
    const uint32_t space = (uint32_t)(ctx->cand ? ctx->n_cand : ctx->n);
    ProfScope prof(ctx->ex, LP_PROF_NEGATIVES, (double)B * k * 8.0);
    unsigned long long *counter = ctx->exhausted_dev + ctx->neg_calls % 16, *next = ctx->exhausted_dev + (ctx->neg_calls + 1) % 16;
    ctx->neg_calls += 1;
    launch_dep(sample_negatives_kernel, dim3(nblk(B * k)), dim3(256), 0, ctx->ex.st, ctx->n, ctx->rowptr, ctx->col, ctx->cand, space,
               make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)), (uint32_t)step, k, mode, reject, attempts, pos_src, B, edge_index_base, neg_src, neg_dst,
               counter, next);
    ctx->ex.launches += 1;
    CK_LAUNCH();
    return LP_OK;
}

// ----------------------------------------------------------------------------------------------
// the step
// ----------------------------------------------------------------------------------------------
template <typename T> static T *tptr(void *p) { return (T *)p; }

// BF16 path: the weight matrices of the flat parameter vector, as the kernels that make its BF16 copies need them
static WeightBlocks weight_blocks(const lp_ctx *ctx)
{
    WeightBlocks wb{};
    for (int k = 0; k < ctx->K; ++k) {
        wb.off[wb.count] = ctx->layer[k].off_w; wb.kin[wb.count] = ctx->layer[k].Kin; wb.fo[wb.count] = ctx->layer[k].Fo;
        wb.split[wb.count] = ctx->cat_grad[k] ? ctx->layer[k].Fi : 0;
        ++wb.count;
    }
    if (ctx->mlp)
        for (int j = 0; j < 2; ++j) { wb.off[wb.count] = ctx->pred[j].off_w; wb.kin[wb.count] = ctx->pred[j].Kin; wb.fo[wb.count] = ctx->pred[j].Fo; ++wb.count; }
    return wb;
}
// one launch turns the call's parameter vector into the BF16 copies the transforms read (lp_score; a training step does it in its first kernel)
static void cache_weights(lp_ctx *ctx, const float *params)
{
    if (ctx->desc.prec != LP_BF16 || !ctx->w16) return;
    launch_dep(weights_cache_kernel, dim3(nblk(ctx->n_params)), dim3(256), 0, ctx->ex.st, params, ctx->n_params, weight_blocks(ctx), ctx->w16, ctx->w16t, ctx->w16s);
    ctx->ex.launches += 1;
}

// dense transform of one layer: Out = act(A W + b)
template <typename T>
static lp_status layer_linear(lp_ctx *ctx, int64_t rows, const LayerBuf &L, const float *params, T *out, int ldo, bool relu, uint32_t *sign_bits = nullptr)
{
    if (rows <= 0) return LP_OK;
    ProfScope prof(ctx->ex, LP_PROF_GEMM_FWD, gemm_bytes((double)rows, L.Fo, L.Kin, sizeof(T), sizeof(T)), 2.0 * rows * L.Fo * L.Kin);
    if (sizeof(T) == 2 && tc_linear_supported(L.Kin, L.Fo)) {
        std::string err;  // Out = A W: the K-major GEMM reads W^T [Fo, Kin] from the transposed BF16 copy
        if (!tc_gemm_kmajor(ctx->tc, ctx->ex, rows, L.Fo, L.Kin, (const bf16 *)L.A, L.Kin, ctx->w16t + L.off_w, params + L.off_b, relu, (bf16 *)out, ldo, err, nullptr, 0,
                            sign_bits))
            return fail(ctx, LP_ECUDA, "tensor-core GEMM: " + err);
        return LP_OK;
    }
    if (sign_bits) return fail(ctx, LP_ESTATE, "sign-bit words asked of a transform that does not run on the tensor cores");
    gemm_simt<T, float, T, false, true>(ctx->ex, rows, L.Fo, L.Kin, (const T *)L.A, L.Kin, params + L.off_w, L.Fo, out, ldo, params + L.off_b, relu ? 1 : 0);
    return LP_OK;
}

// dA[rows, Kin] = dZ[rows, Fo] * W^T
// dA[rows, Kin] = dZ[rows, Fo] * W^T.  For SAGE-mean the right half of dA (the gradient of the mean) is
// multiplied by row_scale = 1 / |N(v)| on the way out, so the adjoint aggregation needs no per-entry
// coefficient: dH[u] = sum over v with u in N(v) of dA_mean[v] / |N(v)|.
template <typename T>
static lp_status layer_input_grad(lp_ctx *ctx, int64_t rows, const LayerBuf &L, const float *params, const T *dZ, int ldz, T *dA, const float *row_scale,
                                  int scale_col0)
{
    if (rows <= 0) return LP_OK;
    ProfScope prof(ctx->ex, LP_PROF_GEMM_DGRAD, gemm_bytes((double)rows, L.Kin, L.Fo, sizeof(T), sizeof(T)), 2.0 * rows * L.Fo * L.Kin);
    if (sizeof(T) == 2 && tc_linear_supported(L.Fo, L.Kin)) {
        std::string err;  // dA = dZ W^T: W [Kin, Fo] as stored is the [N, K] operand
        if (!tc_gemm_kmajor(ctx->tc, ctx->ex, rows, L.Kin, L.Fo, (const bf16 *)dZ, ldz, ctx->w16 + L.off_w, nullptr, false, (bf16 *)dA, L.Kin, err, row_scale,
                            scale_col0))
            return fail(ctx, LP_ECUDA, "tensor-core GEMM: " + err);
        return LP_OK;
    }
    gemm_simt<T, float, T, false, false>(ctx->ex, rows, L.Kin, L.Fo, dZ, ldz, params + L.off_w, L.Fo, dA, L.Kin, nullptr, 0, row_scale, scale_col0);
    return LP_OK;
}

template <typename T>
static lp_status layer_weight_grad(lp_ctx *ctx, int64_t rows, const LayerBuf &L, const T *dZ, int ldz, float *grads, int accumulate)
{
    if (rows <= 0) {
        if (!accumulate) cudaMemsetAsync(grads + L.off_w, 0, sizeof(float) * ((size_t)L.Kin * L.Fo + L.Fo), ctx->ex.st);
        return LP_OK;
    }
    ProfScope prof(ctx->ex, LP_PROF_GEMM_WGRAD, (double)rows * (L.Kin + 2.0 * L.Fo) * sizeof(T) + 4.0 * (L.Kin + 1.0) * L.Fo, 2.0 * rows * L.Fo * (L.Kin + 1.0));
    if (sizeof(T) == 2 && tc_weight_grad_supported(L.Kin, L.Fo)) {
        std::string err;
        // the bias gradient follows the weights in the flat vector: one launch pair produces both
        const bool fuse_bias = L.off_b == L.off_w + (int64_t)L.Kin * L.Fo;
        if (!tc_weight_grad(ctx->tc, ctx->ex, rows, L.Kin, L.Fo, (const bf16 *)L.A, L.Kin, (const bf16 *)dZ, ldz, grads + L.off_w, accumulate, ctx->partials, err,
                            fuse_bias))
            return fail(ctx, LP_ECUDA, "tensor-core GEMM: " + err);
        if (fuse_bias) return LP_OK;
    } else {
        weight_grad_simt<T>(ctx->ex, rows, L.Kin, L.Fo, (const T *)L.A, L.Kin, dZ, ldz, grads + L.off_w, accumulate, ctx->partials);
    }
    colsum<T>(ctx->ex, dZ, rows, L.Fo, ldz, grads + L.off_b, accumulate, ctx->partials);
    return LP_OK;
}

static lp_status sync_counts(lp_ctx *ctx, const int *dev_a, const int *dev_b, int *out_a, int *out_b)
{
    CK(cudaMemcpyAsync(ctx->host_counts, dev_a, sizeof(int), cudaMemcpyDeviceToHost, ctx->ex.st));
    if (dev_b) CK(cudaMemcpyAsync(ctx->host_counts + 1, dev_b, sizeof(int), cudaMemcpyDeviceToHost, ctx->ex.st));
    CK(cudaStreamSynchronize(ctx->ex.st));
    *out_a = ctx->host_counts[0];
    if (dev_b) *out_b = ctx->host_counts[1];
    return LP_OK;
}

// GCN coefficients of a sampled block (entries and destination self terms); hb.entries and hb.n_dst are known
static void gcn_block_coefficients(lp_ctx *ctx, HopBlock &hb, HopBlock &prev)
{
    cudaStream_t st = ctx->ex.st;
    if (hb.entries > 0)
        launch_dep(gcn_block_coef_kernel, dim3(nblk(hb.entries)), dim3(256), 0, st, ctx->rowptr, prev.frontier, hb.blk_ptr, hb.blk_row, hb.blk_eid, hb.blk_ptr + hb.n_dst,
                                                                ctx->gcn_val, hb.blk_val);
    if (hb.n_dst > 0) launch_dep(gather_by_id_kernel, dim3(nblk(hb.n_dst)), dim3(256), 0, st, ctx->gcn_self, prev.frontier, prev.n_front_dev, hb.cap_dst, hb.self_coef_dst);
    ctx->ex.launches += 2;
}

// Sampled computational graph of the batch: F_0 = unique(seeds); hop h samples fanout[h-1]
// in-neighbours of every node of F_{h-1}; F_h = unique(F_{h-1} u sampled).
static lp_status build_blocks(lp_ctx *ctx, const int *pos_src, const int *pos_dst, int64_t B, const int *neg_src, const int *neg_dst, int k,
                              uint64_t seed, uint64_t step)
{
    cudaStream_t st = ctx->ex.st;
    const int n = ctx->n, K = ctx->K;
    const uint2 key = make_uint2((uint32_t)seed, (uint32_t)(seed >> 32));
    const bool gcn = ctx->desc.arch == LP_GCN;
    ProfScope prof(ctx->ex, LP_PROF_BLOCKS);
    CK(cudaMemsetAsync(ctx->mark, 0, (size_t)n, st));
    launch_dep(mark_ids_kernel, dim3(nblk(B)), dim3(256), 0, st, pos_src, B, n, ctx->mark);
    launch_dep(mark_ids_kernel, dim3(nblk(B)), dim3(256), 0, st, pos_dst, B, n, ctx->mark);
    if (k > 0) launch_dep(mark_ids_kernel, dim3(nblk(B * k)), dim3(256), 0, st, neg_dst, B * k, n, ctx->mark);
    if (k > 0 && neg_src) launch_dep(mark_ids_kernel, dim3(nblk(B * k)), dim3(256), 0, st, neg_src, B * k, n, ctx->mark);
    ctx->ex.launches += 4;
    for (int h = 0; h <= K; ++h) {
        HopBlock &hb = ctx->hop[h];
        if (h >= 1) {
            HopBlock &prev = ctx->hop[h - 1];
            hb.n_dst = prev.n_src;
            // sample: counts -> offsets -> columns (also marks the sampled ids; F_{h-1} is still marked)
            launch_dep(nbr_count_kernel, dim3(nblk(hb.n_dst + 1)), dim3(256), 0, st, ctx->rowptr, prev.frontier, prev.n_front_dev, ctx->desc.fanout[h - 1], hb.blk_ptr, hb.n_dst);
            exclusive_scan_i32(ctx->ex, hb.blk_ptr, hb.n_dst, hb.blk_ptr, hb.blk_ptr + hb.n_dst, ctx->scan_tmp);
            {
                const int fo = ctx->desc.fanout[h - 1];
                const uint32_t st32 = (uint32_t)step, h32 = (uint32_t)h;
                if (fo <= 8)
                    launch_dep(nbr_sample_kernel<8>, dim3(nblk((int64_t)hb.n_dst * 8)), dim3(256), 0, st, ctx->rowptr, ctx->col, prev.frontier, prev.n_front_dev, fo, key, st32, h32,
                                                                                      hb.blk_ptr, hb.blk_col_global, hb.blk_row, ctx->mark, hb.blk_eid);
                else if (fo <= 16)
                    launch_dep(nbr_sample_kernel<16>, dim3(nblk((int64_t)hb.n_dst * 16)), dim3(256), 0, st, ctx->rowptr, ctx->col, prev.frontier, prev.n_front_dev, fo, key, st32, h32,
                                                                                        hb.blk_ptr, hb.blk_col_global, hb.blk_row, ctx->mark, hb.blk_eid);
                else
                    launch_dep(nbr_sample_kernel<32>, dim3(nblk((int64_t)hb.n_dst * 32)), dim3(256), 0, st, ctx->rowptr, ctx->col, prev.frontier, prev.n_front_dev, fo, key, st32, h32,
                                                                                        hb.blk_ptr, hb.blk_col_global, hb.blk_row, ctx->mark, hb.blk_eid);
            }
            launch_dep(inv_degree_kernel, dim3(nblk(hb.n_dst)), dim3(256), 0, st, hb.blk_ptr, hb.n_dst, nullptr, hb.inv_deg);
            ctx->ex.launches += 3;
            if (h == K) {  // outermost hop: only the entry count is needed
                int entries = 0, dummy = 0;
                lp_status s = sync_counts(ctx, hb.blk_ptr + hb.n_dst, nullptr, &entries, &dummy);
                if (s != LP_OK) return s;
                hb.entries = entries;
                hb.n_src = n;
                if (gcn) gcn_block_coefficients(ctx, hb, prev);
                break;
            }
        }
        // frontier F_h from the marks
        launch_dep(mark_to_int_kernel, dim3(nblk(n)), dim3(256), 0, st, ctx->mark, n, ctx->flags);
        exclusive_scan_i32(ctx->ex, ctx->flags, n, hb.posmap, hb.n_front_dev, ctx->scan_tmp);
        launch_dep(compact_frontier_kernel, dim3(nblk(n)), dim3(256), 0, st, ctx->mark, hb.posmap, n, hb.frontier);
        ctx->ex.launches += 2;
        int nf = 0, entries = 0;
        lp_status s = sync_counts(ctx, hb.n_front_dev, h >= 1 ? hb.blk_ptr + hb.n_dst : nullptr, &nf, &entries);
        if (s != LP_OK) return s;
        hb.n_src = nf;
        if (h >= 1) {
            hb.entries = entries;
            // local ids, self positions, transposed block
            launch_dep(fill_i32_kernel, dim3(nblk(hb.n_src)), dim3(256), 0, st, hb.inv_self, hb.n_src, -1);
            launch_dep(self_index_kernel, dim3(nblk(hb.n_dst)), dim3(256), 0, st, ctx->hop[h - 1].frontier, ctx->hop[h - 1].n_front_dev, hb.posmap, hb.self_idx, hb.inv_self);
            ctx->ex.launches += 2;
            if (hb.entries > 0) {
                launch_dep(relabel_kernel, dim3(nblk(hb.entries)), dim3(256), 0, st, hb.blk_col_global, hb.blk_ptr + hb.n_dst, hb.entries, hb.posmap, hb.blk_col_local);
                ctx->ex.launches += 1;
            }
            transpose_csr(ctx->ex, hb.blk_ptr, hb.n_dst, hb.n_src, hb.blk_col_local, hb.entries, hb.colptr, hb.rowidx, hb.perm, ctx->tsp, hb.blk_row);
            if (gcn) {
                gcn_block_coefficients(ctx, hb, ctx->hop[h - 1]);
                if (hb.entries > 0) launch_dep(gather_f32_kernel, dim3(nblk(hb.entries)), dim3(256), 0, st, hb.blk_val, hb.perm, hb.entries, hb.blk_valT);
                launch_dep(gather_by_id_kernel, dim3(nblk(hb.n_src)), dim3(256), 0, st, ctx->gcn_self, hb.frontier, hb.n_front_dev, hb.cap_src, hb.self_coef_src);
                ctx->ex.launches += 2;
            }
        }
    }
    CK_LAUNCH();
    return LP_OK;
}

template <typename T> static lp_status forward_impl(lp_ctx *ctx, const float *params)
{
    const int K = ctx->K;
    const bool sage = ctx->desc.arch == LP_SAGE_MEAN;
    const int n = ctx->n;
    const T *Xt = sizeof(T) == 2 ? (const T *)ctx->X16 : (const T *)ctx->X32;
    for (int k = 0; k < K; ++k) {
        LayerBuf &L = ctx->layer[k];
        SpmmArgs<T> a;
        if (!ctx->sampled) {
            a.heavy = ctx->plan_csr;
            a.nnz = ctx->nnz;
        } else {  // sampled rows hold at most `fanout` (<= 32) entries: never heavy
            a.heavy = ctx->plan_dyn;
            a.heavy.host_rows = 0;
            a.heavy.host_items = 0;
            a.nnz = ctx->hop[K - k].entries;
        }
        int64_t rows;
        T *out;
        int ldo;
        if (!ctx->sampled) {
            rows = n;
            a.n_rows = n;
            a.rowptr = ctx->rowptr;
            a.col = ctx->col;
            a.F = L.Fi;
            if (sage) {
                a.X = tptr<T>(L.A);
                a.ldx = L.Kin;
                a.Y = tptr<T>(L.A) + L.Fi;
                a.ldy = L.Kin;
                a.row_scale = ctx->inv_deg;
            } else {
                a.X = tptr<T>(L.Hin);
                a.ldx = L.Fi;
                a.Y = tptr<T>(L.A);
                a.ldy = L.Fi;
                a.val = ctx->gcn_val;
                a.init = a.X;
                a.ldinit = L.Fi;
                a.init_coef = ctx->gcn_self;
            }
            if (k == K - 1) { out = tptr<T>(ctx->HK); ldo = L.Fo; }
            else if (sage) { out = tptr<T>(ctx->layer[k + 1].A); ldo = ctx->layer[k + 1].Kin; }
            else { out = tptr<T>(ctx->layer[k + 1].Hin); ldo = L.Fo; }
        } else {
            HopBlock &hb = ctx->hop[K - k];
            rows = hb.n_dst;
            a.n_rows = hb.n_dst;
            a.rowptr = hb.blk_ptr;
            a.F = L.Fi;
            a.ldx = L.Fi;
            const int *self_rows;
            if (k == 0) {  // innermost layer reads the feature matrix by global id
                a.X = Xt;
                a.col = hb.blk_col_global;
                self_rows = ctx->hop[K - 1].frontier;
            } else {
                a.X = tptr<T>(ctx->layer[k - 1].Hout);
                a.col = hb.blk_col_local;
                self_rows = hb.self_idx;
            }
            if (sage) {  // [h_v | mean over the sample]
                a.row_scale = hb.inv_deg;
                a.Y = tptr<T>(L.A) + L.Fi;
                a.ldy = L.Kin;
                a.self_out = tptr<T>(L.A);
                a.ldself = L.Kin;
                a.self_idx = self_rows;
            } else {     // h_v / d~_v + rescaled sample with the graph's coefficients
                a.val = hb.blk_val;
                a.Y = tptr<T>(L.A);
                a.ldy = L.Fi;
                a.init = a.X;
                a.ldinit = L.Fi;
                a.init_idx = self_rows;
                a.init_coef = hb.self_coef_dst;
            }
            if (k == K - 1) { out = tptr<T>(ctx->HK); ldo = L.Fo; } else { out = tptr<T>(L.Hout); ldo = L.Fo; }
        }
        const bool cached = (k == 0 && !ctx->sampled && ctx->desc.cache_input_aggregation && ctx->input_agg_valid);
        if (!cached) {
            ProfScope prof(ctx->ex, LP_PROF_AGG_FWD, spmm_bytes(a, ctx->sampled ? ctx->hop[K - k].entries : ctx->nnz), 2.0 * (ctx->sampled ? ctx->hop[K - k].entries : ctx->nnz) * L.Fi);
            if (rows > 0 && !spmm_launch<T>(ctx->ex, a)) return fail(ctx, LP_EUNSUPPORTED, "aggregation width not supported");
            if (k == 0 && !ctx->sampled) ctx->input_agg_valid = true;  // AGG(X) stays in layer 1's operand buffer
        }
        lp_status s = layer_linear<T>(ctx, rows, L, params, out, ldo, k < K - 1, (k < K - 1 && ctx->cat_grad[k + 1]) ? ctx->relu_bits[k + 1] : nullptr);
        if (s != LP_OK) return s;
    }
    ctx->rows_out = ctx->sampled ? ctx->hop[0].n_src : n;
    ctx->have_forward = true;
    ctx->hk_valid = !ctx->sampled;
    ctx->hk_params = params;
    ctx->hk_version = ctx->param_version;
    CK_LAUNCH();
    return LP_OK;
}

// ---- MLP edge predictor ----------------------------------------------------------------------
// scores of the E = B (1 + k) edges (positives, then negatives) into ctx->pred_scores; keeps z0, p1, p2
template <typename T>
static lp_status predictor_forward(lp_ctx *ctx, const float *params, const int *idmap, const int *pos_src, const int *pos_dst, int64_t B,
                                   const int *neg_src, const int *neg_dst, int k)
{
    cudaStream_t st = ctx->ex.st;
    const int D = ctx->desc.dims[ctx->K], Hp = ctx->Hp;
    const int64_t E = B * (1 + (int64_t)k);
    constexpr int VN = Vec16<T>::N;
    const int chunks = D / VN;
    const unsigned blocks = nblk(E, EDGE_THREADS / 32);
    T *Z0 = tptr<T>(ctx->pred[0].A), *P1 = tptr<T>(ctx->pred[1].A), *P2 = tptr<T>(ctx->P2), *HK = tptr<T>(ctx->HK);
    if (chunks <= 32) launch_dep(edge_hadamard_kernel<T, 1>, dim3(blocks), dim3(EDGE_THREADS), 0, st, HK, D, D, ctx->n, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, Z0);
    else if (chunks <= 64) launch_dep(edge_hadamard_kernel<T, 2>, dim3(blocks), dim3(EDGE_THREADS), 0, st, HK, D, D, ctx->n, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, Z0);
    else launch_dep(edge_hadamard_kernel<T, 4>, dim3(blocks), dim3(EDGE_THREADS), 0, st, HK, D, D, ctx->n, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, Z0);
    ctx->ex.launches += 1;
    lp_status s = layer_linear<T>(ctx, E, ctx->pred[0], params, P1, Hp, true);
    if (s != LP_OK) return s;
    s = layer_linear<T>(ctx, E, ctx->pred[1], params, P2, Hp, true);
    if (s != LP_OK) return s;
    launch_dep(edge_gemv_kernel<T>, dim3(blocks), dim3(EDGE_THREADS), 0, st, P2, Hp, E, params + ctx->off_w2, params + ctx->off_b2, ctx->pred_scores);
    ctx->ex.launches += 1;
    CK_LAUNCH();
    return LP_OK;
}

// gradients of the predictor's parameters and dL/dz0 (ctx->dZ0) from the per-edge score gradients g
template <typename T>
static lp_status predictor_backward(lp_ctx *ctx, const float *params, int64_t E, const float *g, float *grads, int accumulate)
{
    cudaStream_t st = ctx->ex.st;
    const int Hp = ctx->Hp;
    T *P1 = tptr<T>(ctx->pred[1].A), *P2 = tptr<T>(ctx->P2), *dPa = tptr<T>(ctx->dPa), *dPb = tptr<T>(ctx->dPb), *dZ0 = tptr<T>(ctx->dZ0);
    // last layer: dw2 = P2^T g, db2 = sum g (two fixed-order stages)
    const int splits = colsum_splits(E);
    const int64_t rpb = ceil_div64(E, splits);
    launch_dep(pred_last_layer_grad_kernel<T>, dim3(splits), dim3(256), 0, st, P2, Hp, E, g, rpb, ctx->partials);
    launch_dep(reduce_partials_short_kernel, dim3(nblk(Hp + 1, 32)), dim3(256), 0, st, ctx->partials, Hp + 1, splits, grads + ctx->off_w2, accumulate);
    launch_dep(pred_out_grad_kernel<T>, dim3(nblk(E * Hp)), dim3(256), 0, st, P2, Hp, E, g, params + ctx->off_w2, dPa);
    ctx->ex.launches += 3;
    lp_status s = layer_weight_grad<T>(ctx, E, ctx->pred[1], dPa, ctx->pred[1].Fo, grads, accumulate);
    if (s != LP_OK) return s;
    s = layer_input_grad<T>(ctx, E, ctx->pred[1], params, dPa, ctx->pred[1].Fo, dPb, nullptr, 0);
    if (s != LP_OK) return s;
    launch_dep(relu_mask_kernel<T>, dim3(nblk(E * Hp)), dim3(256), 0, st, dPb, P1, E * Hp);
    ctx->ex.launches += 1;
    s = layer_weight_grad<T>(ctx, E, ctx->pred[0], dPb, ctx->pred[0].Fo, grads, accumulate);
    if (s != LP_OK) return s;
    s = layer_input_grad<T>(ctx, E, ctx->pred[0], params, dPb, ctx->pred[0].Fo, dZ0, nullptr, 0);
    if (s != LP_OK) return s;
    CK_LAUNCH();
    return LP_OK;
}

template <typename T>
static lp_status train_impl(lp_ctx *ctx, const float *params, const int *pos_src, const int *pos_dst, int64_t B, const int *neg_src, const int *neg_dst,
                            int k, uint64_t seed, uint64_t step, float *loss, float *grads, int accumulate)
{
    cudaStream_t st = ctx->ex.st;
    const int K = ctx->K;
    const bool sage = ctx->desc.arch == LP_SAGE_MEAN;
    const int D = ctx->desc.dims[K];
    ctx->ex.prof.tick += 1;  // lp_profile_sample_every counts training steps
    // bad ids are clamped by every consumer and reported through the context's error word; the same launch clears the step's
    // counters and (BF16 path) makes the BF16 copies of the weights
    {
        const int64_t nk = k > 0 ? B * k : 0;
        const bool w16 = ctx->desc.prec == LP_BF16 && ctx->w16;
        const unsigned id_blocks = nblk(2 * B + 2 * nk), w_blocks = w16 ? nblk(ctx->n_params) : 0u;
        launch_dep(check_step_ids_kernel, dim3(id_blocks + w_blocks), dim3(256), 0, st, pos_src, B, pos_dst, B, neg_dst, nk, neg_src, (k > 0 && neg_src) ? nk : 0, ctx->n,
                   ctx->err_flag, ctx->inc_ptr, ctx->inc_cap, ctx->plan_dyn.counts, (int)id_blocks, params, (long long)ctx->n_params, weight_blocks(ctx), ctx->w16, ctx->w16t,
                   ctx->w16s);
        ctx->ex.launches += 1;
    }
    if (ctx->sampled) {
        lp_status s = build_blocks(ctx, pos_src, pos_dst, B, neg_src, neg_dst, k, seed, step);
        if (s != LP_OK) return s;
    }
    lp_status s = forward_impl<T>(ctx, params);
    if (s != LP_OK) return s;
    const int rows_out = ctx->rows_out;
    const int *idmap = ctx->sampled ? ctx->hop[0].posmap : nullptr;
    const int64_t E = B * (1 + (int64_t)k);
    const float inv_N = 1.f / (float)E;
    T *HK = tptr<T>(ctx->HK);

    // scores, loss, per-edge gradients
    std::unique_ptr<ProfScope> pscore(new ProfScope(ctx->ex, LP_PROF_SCORE, (double)B * (2.0 + k) * D * sizeof(T) + (double)E * 12.0, 2.0 * E * D));
    const unsigned eblocks = nblk(B, EDGE_THREADS / 32);
    constexpr int VN = Vec16<T>::N;
    const int chunks = D / VN;
    const float *g_pos = ctx->g_pos, *g_neg = ctx->g_neg;
    unsigned loss_parts = 0;
    // the dot-product scoring kernel also counts the incidence-list lengths (into the zeroed offsets array)
    // (the offsets array was cleared by the first kernel of the step)
    if (ctx->mlp) {
        s = predictor_forward<T>(ctx, params, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k);
        if (s != LP_OK) return s;
        const unsigned lblocks = nblk(E, 256);
        launch_dep(bce_from_scores_kernel, dim3(lblocks), dim3(256), 0, st, ctx->pred_scores, E, B, inv_N, ctx->g_pos, ctx->loss_partials);
        launch_dep(loss_reduce_kernel, dim3(1), dim3(1024), 0, st, ctx->loss_partials, lblocks, inv_N, loss);
        g_neg = ctx->g_pos + B;  // one array: positives, then negatives
        s = predictor_backward<T>(ctx, params, E, ctx->g_pos, grads, accumulate);
        if (s != LP_OK) return s;
    } else {
        unsigned lparts = eblocks;  // loss partials written
        if (chunks <= 32 && k == 1 && !neg_src) {
            lparts = nblk(B, 2 * (EDGE_THREADS / 32));
            launch_dep(edge_score_bce_pair_kernel<T>, dim3(lparts), dim3(EDGE_THREADS), 0, st, HK, D, D, ctx->n, idmap, pos_src, pos_dst, B, neg_dst, inv_N, ctx->g_pos, ctx->g_neg, ctx->loss_partials, ctx->inc_ptr);
        } else if (chunks <= 32) launch_dep(edge_score_bce_kernel<T, 1>, dim3(eblocks), dim3(EDGE_THREADS), 0, st, HK, D, D, ctx->n, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, inv_N, ctx->g_pos, ctx->g_neg, nullptr, nullptr, ctx->loss_partials, ctx->inc_ptr);
        else if (chunks <= 64) launch_dep(edge_score_bce_kernel<T, 2>, dim3(eblocks), dim3(EDGE_THREADS), 0, st, HK, D, D, ctx->n, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, inv_N, ctx->g_pos, ctx->g_neg, nullptr, nullptr, ctx->loss_partials, ctx->inc_ptr);
        else launch_dep(edge_score_bce_kernel<T, 4>, dim3(eblocks), dim3(EDGE_THREADS), 0, st, HK, D, D, ctx->n, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, inv_N, ctx->g_pos, ctx->g_neg, nullptr, nullptr, ctx->loss_partials, ctx->inc_ptr);
        loss_parts = lparts;  // reduced by a block that rides along with the list fill below
    }
    pscore.reset();
    ctx->ex.launches += ctx->mlp ? 2 : 1;

    // incidence lists of the scored edges, grouped by node (slots claimed with integer atomics)
    std::unique_ptr<ProfScope> pinc(new ProfScope(ctx->ex, LP_PROF_INCIDENCE, (double)E * 2.0 * 24.0));
    if (ctx->mlp) launch_dep(incidence_count_kernel, dim3(nblk(E)), dim3(256), 0, st, ctx->n, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, ctx->inc_ptr);
    exclusive_scan_i32_copy(ctx->ex, ctx->inc_ptr, rows_out, ctx->inc_ptr, ctx->inc_cursor, ctx->inc_ptr + rows_out, ctx->scan_tmp);
    {
        // the same launch builds the heavy-row plan of the lists (their offsets are final after the scan; the plan's counters
        // were cleared by the first kernel of the step) and, for the dot-product predictor, reduces the loss partials
        FillRiders x;
        x.fill_blocks = (int)nblk(E);
        x.plan_rowptr = ctx->inc_ptr;
        x.plan_rows = (int)rows_out;
        x.plan = ctx->plan_dyn;
        if (!ctx->mlp) {
            x.loss_partials = ctx->loss_partials;
            x.n_partials = loss_parts;
            x.inv_N = inv_N;
            x.loss = loss;
        }
        launch_dep(incidence_fill_kernel, dim3(nblk(E) + fill_rider_blocks(x)), dim3(256), 0, st, ctx->n, idmap, pos_src, pos_dst, B, neg_src, neg_dst, k, g_pos, g_neg,
                   ctx->inc_cursor, ctx->inc_col, ctx->mlp ? nullptr : ctx->inc_val, ctx->mlp ? ctx->inc_edge : nullptr, nullptr, x);
    }
    ctx->ex.launches += 2;
    pinc.reset();

    // dL/dH^(K)[v] = sum over incident scored edges of g_e * h_other
    // (a layer that aggregates its gradient before the transform keeps dZ as the left half of a [rows, 2 Fo] operand)
    int cur = 1, cat_cur = 0;
    T *dZ = tptr<T>(ctx->dHK);
    int ldz = D;
    if (K >= 2 && ctx->cat_grad[K - 1]) { dZ = tptr<T>(ctx->dcat[cat_cur]); ldz = 2 * D; }
    ctx->out_grad = dZ;
    ctx->out_grad_ld = ldz;
    {
        SpmmArgs<T> a;
        a.heavy = ctx->plan_dyn;
        a.heavy.partials = ctx->inc_partials;
        a.heavy.plan_prebuilt = true;  // by the launch that filled the lists

        a.nnz = 2 * E;
        a.n_rows = rows_out;
        a.rowptr = ctx->inc_ptr;
        a.col = ctx->inc_col;
        a.X = HK;
        a.ldx = D;
        a.F = D;
        a.Y = dZ;
        a.ldy = ldz;
        if (K >= 2 && ctx->cat_grad[K - 1]) {  // the adjoint of the mean gathers dZ[v] / |N(v)|: written here, beside dZ, so that it needs no coefficients
            a.Y2 = tptr<T>(ctx->dHK);
            a.ldy2 = D;
            a.y2_scale = ctx->inv_deg;
        }
        // Scale of the exact sum.  Every coefficient carries the 1 / N of the mean loss, so the products are of the order
        // |h| / N: the power-of-two scale is 2^s * 2^ceil(log2 N) with s = min(32, 50 - ceil(log2 N)), which resolves a
        // product to 2^-s relative to |h| / N whatever the batch size.  The coefficients of one node add up to at most 1
        // in magnitude (dot product; a small multiple of it behind the MLP), so a node's sum stays below 2^63 as long
        // as the embeddings stay below 4096 in magnitude.
        {
            int lg = 0;
            while (((int64_t)1 << lg) < E) ++lg;
            const int sh = std::min(32, 50 - lg) + lg;
            a.exact_scale = ldexpf(1.f, sh);
            a.exact_inv = ldexpf(1.f, -sh);
        }
        if (ctx->mlp) {  // dL/dh_node = sum over incident edges of dL/dz0[edge] * h_other
            a.X2 = tptr<T>(ctx->dZ0);
            a.ldx2 = D;
            a.col2 = ctx->inc_edge;
        } else {         // dot product: g_e * h_other
            a.val = ctx->inc_val;
        }
        ProfScope prof(ctx->ex, LP_PROF_SCATTER, spmm_bytes(a, 2 * E), 4.0 * E * D);
        // the order of a node's entries is not reproducible, so the sum is taken exactly (64-bit fixed point)
        if (rows_out > 0 && !spmm_launch<T, long long>(ctx->ex, a)) return fail(ctx, LP_EUNSUPPORTED, "embedding width not supported");
    }
    ctx->have_grad = true;

    // backward through the layers
    for (int l = K - 1; l >= 0; --l) {
        LayerBuf &L = ctx->layer[l];
        const int64_t rows = ctx->sampled ? ctx->hop[K - l].n_dst : ctx->n;
        s = layer_weight_grad<T>(ctx, rows, L, dZ, ldz, grads, accumulate);
        if (s != LP_OK) return s;
        if (l == 0) break;
        // where the gradient of this layer's input goes: the next layer down may want it as the left half of its own operand
        T *dZn = tptr<T>(ctx->dZ[cur ^ 1]);
        int ldn = L.Fi;
        if (l >= 2 && ctx->cat_grad[l - 1]) { dZn = tptr<T>(ctx->dcat[cat_cur ^ 1]); ldn = 2 * L.Fi; }
        if (ctx->cat_grad[l]) {
            // dH^(l) = relu'(H^(l)) * ([dZ | A^T (dZ / deg)] [W_self^T ; W_neigh^T]): aggregate first (plain epilogue, no self
            // term), then one transform over both halves with the ReLU mask taken from the forward transform's sign bits
            if constexpr (sizeof(T) == 2) {
                SpmmArgs<T> a;
                a.heavy = ctx->plan_csc;
                a.nnz = ctx->nnz;
                a.n_rows = ctx->n;
                a.rowptr = ctx->colptr;
                a.col = ctx->rowidx;
                a.F = L.Fo;
                if (l == K - 1) {  // the top layer's dZ / |N(v)| was written beside dZ
                    a.X = tptr<T>(ctx->dHK);
                    a.ldx = L.Fo;
                } else {           // below it the mean's coefficients ride with the entries
                    a.val = ctx->meanT_val;
                    a.X = dZ;
                    a.ldx = ldz;
                }
                a.Y = dZ + L.Fo;
                a.ldy = ldz;
                {
                    ProfScope prof(ctx->ex, LP_PROF_AGG_BWD, spmm_bytes(a, ctx->nnz), 2.0 * ctx->nnz * L.Fo);
                    if (!spmm_launch<T>(ctx->ex, a)) return fail(ctx, LP_EUNSUPPORTED, "aggregation width not supported");
                }
                ProfScope prof(ctx->ex, LP_PROF_GEMM_DGRAD, gemm_bytes((double)rows, L.Fi, 2 * L.Fo, sizeof(T), sizeof(T)), 4.0 * rows * L.Fo * L.Fi);
                std::string err;
                if (!tc_gemm_kmajor(ctx->tc, ctx->ex, rows, L.Fi, 2 * L.Fo, (const bf16 *)dZ, ldz, ctx->w16s + L.off_w, nullptr, false, (bf16 *)dZn, ldn, err, nullptr, 0,
                                    nullptr, ctx->relu_bits[l]))
                    return fail(ctx, LP_ECUDA, "tensor-core GEMM: " + err);
            }
            dZ = dZn;
            ldz = ldn;
            if (l >= 2 && ctx->cat_grad[l - 1]) cat_cur ^= 1; else cur ^= 1;
            continue;
        }
        T *dA = tptr<T>(ctx->dA);
        const float *mean_scale = sage ? (ctx->sampled ? ctx->hop[K - l].inv_deg : ctx->inv_deg) : nullptr;
        s = layer_input_grad<T>(ctx, rows, L, params, dZ, ldz, dA, mean_scale, L.Fi);
        if (s != LP_OK) return s;
        SpmmArgs<T> a;
        if (!ctx->sampled) {
            a.heavy = ctx->plan_csc;
            a.nnz = ctx->nnz;
        } else {
            a.heavy = ctx->plan_dyn;
            a.nnz = ctx->hop[K - l].entries;
        }
        a.F = L.Fi;
        a.Y = dZn;
        a.ldy = ldn;
        if (!ctx->sampled) {
            a.n_rows = ctx->n;
            a.rowptr = ctx->colptr;
            a.col = ctx->rowidx;
            if (sage) {
                a.X = dA + L.Fi;
                a.ldx = L.Kin;
                a.init = dA;
                a.ldinit = L.Kin;
                a.relu_ref = tptr<T>(L.A);  // left half = H^(l)
                a.ldref = L.Kin;
            } else {
                a.val = ctx->gcn_valT;
                a.X = dA;
                a.ldx = L.Fi;
                a.init = dA;
                a.ldinit = L.Fi;
                a.init_coef = ctx->gcn_self;
                a.relu_ref = tptr<T>(L.Hin);
                a.ldref = L.Fi;
            }
        } else {
            HopBlock &hb = ctx->hop[K - l];
            a.n_rows = hb.n_src;
            a.rowptr = hb.colptr;
            a.col = hb.rowidx;
            a.init = dA;
            a.ldinit = L.Kin;
            a.init_idx = hb.inv_self;
            if (sage) {
                a.X = dA + L.Fi;
                a.ldx = L.Kin;
            } else {
                a.val = hb.blk_valT;
                a.X = dA;
                a.ldx = L.Fi;
                a.init_coef = hb.self_coef_src;
            }
            a.relu_ref = tptr<T>(ctx->layer[l - 1].Hout);
            a.ldref = L.Fi;
        }
        {
            const int64_t nnz_l = ctx->sampled ? ctx->hop[K - l].entries : ctx->nnz;
            ProfScope prof(ctx->ex, LP_PROF_AGG_BWD, spmm_bytes(a, nnz_l), 2.0 * nnz_l * L.Fi);
            if (a.n_rows > 0 && !spmm_launch<T>(ctx->ex, a)) return fail(ctx, LP_EUNSUPPORTED, "aggregation width not supported");
        }
        dZ = dZn;
        ldz = ldn;
        if (l >= 2 && ctx->cat_grad[l - 1]) cat_cur ^= 1; else cur ^= 1;
    }
    CK_LAUNCH();
    return LP_OK;
}

static lp_status check_step_args(lp_ctx *ctx, const char *who, const void *params, const void *a, const void *b, int64_t B, const void *neg_dst, int k)
{
    if (!ctx->model_set) return fail(ctx, LP_ESTATE, std::string(who) + ": set a model first");
    if (!params) return fail(ctx, LP_EINVAL, std::string(who) + ": params is NULL");
    if (B <= 0 || B > ctx->max_batch) return fail(ctx, LP_EINVAL, std::string(who) + ": B must be in [1, max_batch]");
    if (k < 0 || k > ctx->max_k) return fail(ctx, LP_EINVAL, std::string(who) + ": k must be in [0, max_k]");
    if (!a || !b) return fail(ctx, LP_EINVAL, std::string(who) + ": edge arrays are NULL");
    if (k > 0 && !neg_dst) return fail(ctx, LP_EINVAL, std::string(who) + ": neg_dst is NULL");
    return LP_OK;
}

extern "C" lp_status lp_train_step(lp_ctx *ctx, const float *params, const int32_t *pos_src, const int32_t *pos_dst, int64_t B,
                                   const int32_t *neg_src, const int32_t *neg_dst, int32_t k, uint64_t seed, uint64_t step, float *loss,
                                   float *grads, int32_t accumulate)
{
    if (!ctx) return LP_EINVAL;
    lp_status s = check_step_args(ctx, "lp_train_step", params, pos_src, pos_dst, B, neg_dst, k);
    if (s != LP_OK) return s;
    if (!loss || !grads) return fail(ctx, LP_EINVAL, "lp_train_step: loss or grads is NULL");
    CK(cudaSetDevice(ctx->device));
    if (ctx->desc.prec == LP_BF16) s = train_impl<bf16>(ctx, params, pos_src, pos_dst, B, neg_src, neg_dst, k, seed, step, loss, grads, accumulate);
    else s = train_impl<float>(ctx, params, pos_src, pos_dst, B, neg_src, neg_dst, k, seed, step, loss, grads, accumulate);
    if (s != LP_OK) return s;
    return tc_check(ctx->tc, ctx->ex, false, ctx->err);
}

extern "C" lp_status lp_adam_step(lp_ctx *ctx, float *params, float *adam_m, float *adam_v, const float *grads, double grad_scale, double lr,
                                  double beta1, double beta2, double eps, int64_t t)
{
    if (!ctx) return LP_EINVAL;
    if (!ctx->model_set) return fail(ctx, LP_ESTATE, "lp_adam_step: set a model first");
    if (!params || !grads) return fail(ctx, LP_EINVAL, "lp_adam_step: params or grads is NULL");
    if ((adam_m == nullptr) != (adam_v == nullptr)) return fail(ctx, LP_EINVAL, "lp_adam_step: pass both moment arrays or neither");
    if (adam_m && t < 1) return fail(ctx, LP_EINVAL, "lp_adam_step: t counts from 1");
    CK(cudaSetDevice(ctx->device));
    const int64_t np = ctx->n_params;
    ctx->param_version += 1;  // embeddings kept for lp_score belong to the old weights
    ProfScope prof(ctx->ex, LP_PROF_ADAM, (double)np * (adam_m ? 28.0 : 12.0));
    if (adam_m) {
        const double c1 = 1.0 - std::pow(beta1, (double)t), c2 = 1.0 - std::pow(beta2, (double)t);
        launch_dep(adam_kernel, dim3(nblk(np)), dim3(256), 0, ctx->ex.st, params, adam_m, adam_v, grads, np, (float)grad_scale, (float)lr, (float)beta1, (float)(1.0 - beta1),
                                                      (float)beta2, (float)(1.0 - beta2), (float)eps, (float)(1.0 / c1), (float)(1.0 / c2));
    } else {
        launch_dep(sgd_kernel, dim3(nblk(np)), dim3(256), 0, ctx->ex.st, params, grads, np, (float)grad_scale, (float)lr);
    }
    ctx->ex.launches += 1;
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_train_step_host(lp_ctx *ctx, float *params, const int32_t *pos_src_host, const int32_t *pos_dst_host, int64_t B, int32_t k,
                                        uint64_t seed, uint64_t step, int64_t edge_index_base, float *adam_m, float *adam_v, int64_t adam_t,
                                        float *loss_host, float *grads_host)
{
    if (!ctx) return LP_EINVAL;
    lp_status s = check_step_args(ctx, "lp_train_step_host", params, pos_src_host, pos_dst_host, B, (const void *)1, k);
    if (s != LP_OK) return s;
    if (!loss_host) return fail(ctx, LP_EINVAL, "lp_train_step_host: loss_host is NULL");
    CK(cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->ex.st;
    int *ps = ctx->d_pos_tmp, *pd = ctx->d_pos_tmp + ctx->max_batch;
    CK(cudaMemcpyAsync(ps, pos_src_host, sizeof(int) * (size_t)B, cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(pd, pos_dst_host, sizeof(int) * (size_t)B, cudaMemcpyHostToDevice, st));
    if (k > 0) {
        s = lp_sample_negatives(ctx, seed, step, k, LP_NEG_PER_SOURCE, ps, B, edge_index_base, nullptr, ctx->d_neg_tmp);
        if (s != LP_OK) return s;
    }
    s = lp_train_step(ctx, params, ps, pd, B, nullptr, ctx->d_neg_tmp, k, seed, step, ctx->d_loss_tmp, ctx->d_grads_tmp, 0);
    if (s != LP_OK) return s;
    if (adam_m || adam_v) {
        s = lp_adam_step(ctx, params, adam_m, adam_v, ctx->d_grads_tmp, 1.0, 1e-3, 0.9, 0.999, 1e-8, adam_t);
        if (s != LP_OK) return s;
    }
    CK(cudaMemcpyAsync(loss_host, ctx->d_loss_tmp, sizeof(float), cudaMemcpyDeviceToHost, st));
    if (grads_host) CK(cudaMemcpyAsync(grads_host, ctx->d_grads_tmp, sizeof(float) * (size_t)ctx->n_params, cudaMemcpyDeviceToHost, st));
    // both error words travel with the loss: one synchronise for the whole call (the words land in pinned memory)
    int *bad = ctx->host_counts + 32;
    *bad = 0;
    CK(cudaMemcpyAsync(bad, ctx->err_flag, sizeof(int), cudaMemcpyDeviceToHost, st));
    const bool tc_asked = tc_check_enqueue(ctx->tc, ctx->ex);
    CK(cudaStreamSynchronize(st));
    if (*bad) {
        cudaMemsetAsync(ctx->err_flag, 0, sizeof(int), st);
        if (*bad & 2) return fail(ctx, LP_ETIMEOUT, "lp_train_step_host: a bounded wait inside the scan of the step expired");
        return fail(ctx, LP_EINVAL, "lp_train_step_host: a node id is outside [0, n)");
    }
    return tc_asked ? tc_check_result(ctx->tc, ctx->ex, ctx->err) : LP_OK;
}

template <typename T>
static lp_status score_impl(lp_ctx *ctx, const float *params, const int *src, const int *dst, int64_t E, uint64_t seed, uint64_t step, float *scores)
{
    if (ctx->sampled) {
        lp_status s = build_blocks(ctx, src, dst, E, nullptr, nullptr, 0, seed, step);
        if (s != LP_OK) return s;
    }
    // full-graph models: H^(K) of the last forward pass is reused while the caller passes the same parameter vector and no
    // call of this library has updated it since
    lp_status s = LP_OK;
    const bool reuse = ctx->hk_valid && ctx->hk_params == params && ctx->hk_version == ctx->param_version;
    if (!reuse || ctx->mlp) cache_weights(ctx, params);  // (the MLP predictor's layers need their weights in any case)
    if (!reuse) s = forward_impl<T>(ctx, params);
    if (s != LP_OK) return s;
    const int D = ctx->desc.dims[ctx->K];
    const int *idmap = ctx->sampled ? ctx->hop[0].posmap : nullptr;
    constexpr int VN = Vec16<T>::N;
    const int chunks = D / VN;
    if (ctx->mlp) {  // in pieces of at most the predictor's buffer size
        const int64_t cap = ctx->max_batch * (1 + (int64_t)ctx->max_k);
        for (int64_t off = 0; off < E; off += cap) {
            const int64_t m = std::min<int64_t>(cap, E - off);
            s = predictor_forward<T>(ctx, params, idmap, src + off, dst + off, m, nullptr, nullptr, 0);
            if (s != LP_OK) return s;
            CK(cudaMemcpyAsync(scores + off, ctx->pred_scores, sizeof(float) * (size_t)m, cudaMemcpyDeviceToDevice, ctx->ex.st));
        }
        return LP_OK;
    }
    const unsigned blocks = nblk(E, EDGE_THREADS / 32);
    if (chunks <= 32) launch_dep(edge_score_kernel<T, 1>, dim3(blocks), dim3(EDGE_THREADS), 0, ctx->ex.st, tptr<T>(ctx->HK), D, D, ctx->n, idmap, src, dst, E, scores);
    else if (chunks <= 64) launch_dep(edge_score_kernel<T, 2>, dim3(blocks), dim3(EDGE_THREADS), 0, ctx->ex.st, tptr<T>(ctx->HK), D, D, ctx->n, idmap, src, dst, E, scores);
    else launch_dep(edge_score_kernel<T, 4>, dim3(blocks), dim3(EDGE_THREADS), 0, ctx->ex.st, tptr<T>(ctx->HK), D, D, ctx->n, idmap, src, dst, E, scores);
    ctx->ex.launches += 1;
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_score(lp_ctx *ctx, const float *params, const int32_t *src, const int32_t *dst, int64_t E, uint64_t seed, uint64_t step,
                              float *scores)
{
    if (!ctx) return LP_EINVAL;
    if (!ctx->model_set) return fail(ctx, LP_ESTATE, "lp_score: set a model first");
    if (!params || !src || !dst || !scores) return fail(ctx, LP_EINVAL, "lp_score: null array");
    if (E <= 0) return fail(ctx, LP_EINVAL, "lp_score: E must be positive");
    if (ctx->sampled && E > ctx->max_batch) return fail(ctx, LP_EINVAL, "lp_score: sampled models score at most max_batch pairs per call");
    CK(cudaSetDevice(ctx->device));
    lp_status s = ctx->desc.prec == LP_BF16 ? score_impl<bf16>(ctx, params, src, dst, E, seed, step, scores)
                                            : score_impl<float>(ctx, params, src, dst, E, seed, step, scores);
    if (s != LP_OK) return s;
    return tc_check(ctx->tc, ctx->ex, false, ctx->err);
}

extern "C" lp_status lp_invalidate_embeddings(lp_ctx *ctx)
{
    if (!ctx) return LP_EINVAL;
    ctx->hk_valid = false;
    return LP_OK;
}

extern "C" lp_status lp_set_wait_limit(lp_ctx *ctx, uint64_t limit_ns, int32_t overdeclare_bytes)
{
    if (!ctx) return LP_EINVAL;
    if (limit_ns < 1000 || limit_ns > 60000000000ull) return fail(ctx, LP_EINVAL, "lp_set_wait_limit: limit must be between 1 us and 60 s");
    if (overdeclare_bytes < 0 || overdeclare_bytes > 65536 || overdeclare_bytes % 16 != 0)
        return fail(ctx, LP_EINVAL, "lp_set_wait_limit: overdeclare_bytes must be a multiple of 16 in [0, 65536]");
    ctx->tc.wait_limit_ns = limit_ns;
    ctx->tc.overdeclare_tx = overdeclare_bytes;
    return LP_OK;
}

extern "C" lp_status lp_hits_at_k(lp_ctx *ctx, const float *pos_scores, int64_t n_pos, const float *neg_scores, int64_t n_neg, int64_t K, double *hits)
{
    if (!ctx || !hits) return LP_EINVAL;
    if (!pos_scores || n_pos <= 0 || (n_neg > 0 && !neg_scores) || n_neg < 0 || K <= 0 || n_neg >= ((int64_t)1 << 31))
        return fail(ctx, LP_EINVAL, "lp_hits_at_k: bad argument");
    if (n_neg < K) { *hits = 1.0; return LP_OK; }
    CK(cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->ex.st;
    std::vector<void *> tmp;
    int64_t tmp_bytes = 0;
    uint32_t *keys = nullptr, *vals = nullptr;
    unsigned long long *count = nullptr;
    SortScratch sc;
    cudaError_t e = dev_alloc(ctx, tmp, tmp_bytes, &keys, n_neg);
    if (e == cudaSuccess) e = dev_alloc(ctx, tmp, tmp_bytes, &vals, n_neg);
    if (e == cudaSuccess) e = dev_alloc(ctx, tmp, tmp_bytes, &sc.keys_alt, n_neg);
    if (e == cudaSuccess) e = dev_alloc(ctx, tmp, tmp_bytes, &sc.vals_alt, n_neg);
    if (e == cudaSuccess) e = dev_alloc(ctx, tmp, tmp_bytes, &sc.hist, SortScratch::hist_ints(n_neg));
    if (e == cudaSuccess) e = dev_alloc(ctx, tmp, tmp_bytes, &sc.scan_tmp, SortScratch::scan_ints(n_neg));
    if (e == cudaSuccess) e = dev_alloc(ctx, tmp, tmp_bytes, &count, 8);
    if (e != cudaSuccess) { free_list(tmp); CK(e); }
    launch_dep(float_keys_kernel, dim3(nblk(n_neg)), dim3(256), 0, st, neg_scores, n_neg, keys, vals);
    const bool in_place = radix_sort_pairs(ctx->ex, keys, vals, n_neg, 32, sc);  // ascending
    cudaMemsetAsync(count, 0, sizeof(unsigned long long), st);
    launch_dep(count_above_kernel, dim3(nblk(n_pos)), dim3(256), 0, st, pos_scores, n_pos, in_place ? keys : sc.keys_alt, n_neg - K, count);
    ctx->ex.launches += 2;
    unsigned long long h = 0;
    e = cudaMemcpyAsync(&h, count, sizeof h, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    free_list(tmp);
    CK(e);
    CK_LAUNCH();
    *hits = (double)h / (double)n_pos;
    return LP_OK;
}

// ----------------------------------------------------------------------------------------------
// inspection
// ----------------------------------------------------------------------------------------------
template <typename T> static void to_f32(lp_ctx *ctx, const T *src, int64_t lds, float *dst, int64_t rows, int F)
{
    if (rows <= 0) return;
    launch_dep(copy_rows_kernel<T, float>, dim3(nblk(rows * F)), dim3(256), 0, ctx->ex.st, src, lds, dst, F, rows, F);
    ctx->ex.launches += 1;
}

extern "C" lp_status lp_get_embeddings(lp_ctx *ctx, int32_t layer, float *out)
{
    if (!ctx || !out) return LP_EINVAL;
    if (!ctx->model_set || !ctx->have_forward) return fail(ctx, LP_ESTATE, "lp_get_embeddings: run a forward pass first");
    const int K = ctx->K;
    if (layer < 1 || layer > K) return fail(ctx, LP_EINVAL, "lp_get_embeddings: layer must be in [1, K]");
    CK(cudaSetDevice(ctx->device));
    const bool b16 = ctx->desc.prec == LP_BF16;
    const int F = ctx->desc.dims[layer];
    const void *src;
    int64_t ld, rows;
    if (layer == K) { src = ctx->HK; ld = F; rows = ctx->rows_out; }
    else if (ctx->sampled) { src = ctx->layer[layer - 1].Hout; ld = F; rows = ctx->hop[K - layer + 1].n_dst; }
    else if (ctx->desc.arch == LP_SAGE_MEAN) { src = ctx->layer[layer].A; ld = ctx->layer[layer].Kin; rows = ctx->n; }
    else { src = ctx->layer[layer].Hin; ld = F; rows = ctx->n; }
    if (b16) to_f32<bf16>(ctx, (const bf16 *)src, ld, out, rows, F); else to_f32<float>(ctx, (const float *)src, ld, out, rows, F);
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_get_predictor_activations(lp_ctx *ctx, int32_t layer, int64_t E, float *out)
{
    if (!ctx || !out) return LP_EINVAL;
    if (!ctx->model_set || !ctx->mlp || !ctx->have_forward) return fail(ctx, LP_ESTATE, "lp_get_predictor_activations: no MLP predictor pass has run");
    if (layer < 1 || layer > 2 || E <= 0 || E > ctx->max_batch * (1 + (int64_t)ctx->max_k)) return fail(ctx, LP_EINVAL, "lp_get_predictor_activations: bad layer or E");
    CK(cudaSetDevice(ctx->device));
    const void *src = layer == 1 ? ctx->pred[1].A : ctx->P2;
    if (ctx->desc.prec == LP_BF16) to_f32<bf16>(ctx, (const bf16 *)src, ctx->Hp, out, E, ctx->Hp);
    else to_f32<float>(ctx, (const float *)src, ctx->Hp, out, E, ctx->Hp);
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_get_output_gradient(lp_ctx *ctx, float *out)
{
    if (!ctx || !out) return LP_EINVAL;
    if (!ctx->model_set || !ctx->have_grad) return fail(ctx, LP_ESTATE, "lp_get_output_gradient: run lp_train_step first");
    CK(cudaSetDevice(ctx->device));
    const int D = ctx->desc.dims[ctx->K];
    if (ctx->desc.prec == LP_BF16) to_f32<bf16>(ctx, (const bf16 *)ctx->out_grad, ctx->out_grad_ld, out, ctx->rows_out, D);
    else to_f32<float>(ctx, (const float *)ctx->out_grad, ctx->out_grad_ld, out, ctx->rows_out, D);
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_get_block(lp_ctx *ctx, int32_t hop, int32_t *frontier, int64_t *blk_ptr, int32_t *blk_col)
{
    if (!ctx) return LP_EINVAL;
    if (!ctx->model_set || !ctx->sampled || !ctx->have_forward) return fail(ctx, LP_ESTATE, "lp_get_block: no sampled step has run");
    if (hop < 0 || hop > ctx->K) return fail(ctx, LP_EINVAL, "lp_get_block: hop out of range");
    CK(cudaSetDevice(ctx->device));
    HopBlock &hb = ctx->hop[hop];
    cudaStream_t st = ctx->ex.st;
    if (frontier) {
        if (hop == ctx->K) return fail(ctx, LP_EUNSUPPORTED, "lp_get_block: the outermost frontier is not materialised (use the block columns)");
        if (hb.n_src > 0) CK(cudaMemcpyAsync(frontier, hb.frontier, sizeof(int) * (size_t)hb.n_src, cudaMemcpyDeviceToDevice, st));
    }
    if (hop >= 1) {
        if (blk_ptr) launch_dep(widen_i32_kernel, dim3(nblk(hb.n_dst + 1)), dim3(256), 0, st, hb.blk_ptr, hb.n_dst + 1, blk_ptr);
        if (blk_col && hb.entries > 0) CK(cudaMemcpyAsync(blk_col, hb.blk_col_global, sizeof(int) * (size_t)hb.entries, cudaMemcpyDeviceToDevice, st));
    }
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_get_stats(lp_ctx *ctx, lp_stats *out)
{
    if (!ctx || !out) return LP_EINVAL;
    CK(cudaSetDevice(ctx->device));
    memset(out, 0, sizeof *out);
    unsigned long long ex = 0;
    int bad = 0;
    CK(cudaMemcpyAsync(&ex, ctx->exhausted_dev + (ctx->neg_calls + 15) % 16, sizeof ex, cudaMemcpyDeviceToHost, ctx->ex.st));  // the last call's counter
    CK(cudaMemcpyAsync(&bad, ctx->err_flag, sizeof bad, cudaMemcpyDeviceToHost, ctx->ex.st));
    CK(cudaStreamSynchronize(ctx->ex.st));
    if (bad) {
        cudaMemsetAsync(ctx->err_flag, 0, sizeof(int), ctx->ex.st);
        if (bad & 2) return fail(ctx, LP_ETIMEOUT, "a bounded wait inside the scan of an earlier step expired (results of that call are invalid)");
        return fail(ctx, LP_EINVAL, "a node id outside [0, n) was passed to an earlier call (it was clamped; results of that call are invalid)");
    }
    out->negatives_exhausted = (int64_t)ex;
    if (ctx->model_set && ctx->sampled) {
        for (int h = 0; h <= ctx->K; ++h) out->block_nodes[h] = ctx->hop[h].n_src;
        for (int h = 1; h <= ctx->K; ++h) out->block_edges[h - 1] = ctx->hop[h].entries;
    }
    out->workspace_bytes = ctx->graph_bytes + ctx->model_bytes;
    out->kernel_launches = ctx->ex.launches;
    return tc_check(ctx->tc, ctx->ex, true, ctx->err);
}

extern "C" lp_status lp_profile_begin(lp_ctx *ctx, uint32_t category_mask)
{
    if (!ctx) return LP_EINVAL;
    CK(cudaSetDevice(ctx->device));
    CK(cudaStreamSynchronize(ctx->ex.st));
    ctx->ex.prof.spans.clear();
    ctx->ex.prof.used = 0;
    ctx->ex.prof.mask = category_mask & ((1u << LP_PROF_CATEGORIES) - 1u);
    return LP_OK;
}

extern "C" lp_status lp_profile_sample_every(lp_ctx *ctx, uint32_t n)
{
    if (!ctx) return LP_EINVAL;
    if (n == 0) return fail(ctx, LP_EINVAL, "lp_profile_sample_every: n must be at least 1");
    ctx->ex.prof.period = n;
    return LP_OK;
}

extern "C" lp_status lp_profile_end(lp_ctx *ctx, lp_profile *out)
{
    if (!ctx || !out) return LP_EINVAL;
    CK(cudaSetDevice(ctx->device));
    ctx->ex.prof.mask = 0;
    CK(cudaStreamSynchronize(ctx->ex.st));
    memset(out, 0, sizeof *out);
    for (const Profiler::Span &s : ctx->ex.prof.spans) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, s.a, s.b) != cudaSuccess) continue;
        out->ms[s.cat] += ms;
        out->bytes[s.cat] += s.bytes;
        out->flops[s.cat] += s.flops;
        out->spans[s.cat] += 1;
    }
    ctx->ex.prof.spans.clear();
    ctx->ex.prof.used = 0;
    return LP_OK;
}

// ----------------------------------------------------------------------------------------------
// single operators
// ----------------------------------------------------------------------------------------------
template <typename T> static lp_status op_aggregate_impl(lp_ctx *ctx, int arch, int transpose, const T *H, int F, T *M)
{
    SpmmArgs<T> a;
    a.heavy = transpose ? ctx->plan_csc : ctx->plan_csr;
    a.nnz = ctx->nnz;
    a.n_rows = ctx->n;
    a.X = H;
    a.ldx = F;
    a.F = F;
    a.Y = M;
    a.ldy = F;
    if (!transpose) {
        a.rowptr = ctx->rowptr;
        a.col = ctx->col;
        if (arch == LP_GCN) { a.val = ctx->gcn_val; a.init = H; a.ldinit = F; a.init_coef = ctx->gcn_self; }
        else a.row_scale = ctx->inv_deg;
    } else {
        a.rowptr = ctx->colptr;
        a.col = ctx->rowidx;
        if (arch == LP_GCN) { a.val = ctx->gcn_valT; a.init = H; a.ldinit = F; a.init_coef = ctx->gcn_self; }
        else a.val = ctx->meanT_val;
    }
    ProfScope prof(ctx->ex, transpose ? LP_PROF_AGG_BWD : LP_PROF_AGG_FWD, spmm_bytes(a, ctx->nnz), 2.0 * ctx->nnz * F);
    if (!spmm_launch<T>(ctx->ex, a)) return fail(ctx, LP_EINVAL, "lp_op_aggregate: F must be a multiple of 8, at most 512");
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_op_aggregate(lp_ctx *ctx, int32_t arch, int32_t transpose, int32_t is_bf16, const void *H, int32_t F, void *M)
{
    if (!ctx) return LP_EINVAL;
    if (!ctx->loaded) return fail(ctx, LP_ESTATE, "lp_op_aggregate: no graph loaded");
    if (!H || !M || H == M) return fail(ctx, LP_EINVAL, "lp_op_aggregate: H and M must be distinct non-null arrays");
    if (arch != LP_GCN && arch != LP_SAGE_MEAN) return fail(ctx, LP_EINVAL, "lp_op_aggregate: unknown architecture");
    if (F <= 0 || F % 8 != 0 || F > 512) return fail(ctx, LP_EINVAL, "lp_op_aggregate: F must be a multiple of 8, at most 512");
    CK(cudaSetDevice(ctx->device));
    return is_bf16 ? op_aggregate_impl<bf16>(ctx, arch, transpose, (const bf16 *)H, F, (bf16 *)M)
                   : op_aggregate_impl<float>(ctx, arch, transpose, (const float *)H, F, (float *)M);
}

extern "C" lp_status lp_op_gather_ceiling(lp_ctx *ctx, int32_t transpose, const void *H, int32_t row_bytes, void *folds)
{
    if (!ctx) return LP_EINVAL;
    if (!ctx->loaded) return fail(ctx, LP_ESTATE, "lp_op_gather_ceiling: no graph loaded");
    if (!H || !folds) return fail(ctx, LP_EINVAL, "lp_op_gather_ceiling: H and folds must be non-null");
    if (row_bytes != 128 && row_bytes != 256 && row_bytes != 512) return fail(ctx, LP_EINVAL, "lp_op_gather_ceiling: row_bytes must be 128, 256 or 512");
    if (((uintptr_t)H & 15) != 0 || ((uintptr_t)folds & 15) != 0) return fail(ctx, LP_EINVAL, "lp_op_gather_ceiling: H and folds must be 16-byte aligned");
    CK(cudaSetDevice(ctx->device));
    gather_probe_launch(ctx->ex, transpose ? ctx->rowidx : ctx->col, ctx->nnz, H, row_bytes, folds);
    CK_LAUNCH();
    return LP_OK;
}

extern "C" lp_status lp_op_linear(lp_ctx *ctx, int32_t prec, int64_t M, int32_t N, int32_t K, const void *A, const void *B, int32_t trans_b,
                                  const float *bias, int32_t relu, void *C)
{
    if (!ctx) return LP_EINVAL;
    if (!A || !B || !C || M <= 0 || N <= 0 || K <= 0) return fail(ctx, LP_EINVAL, "lp_op_linear: bad argument");
    CK(cudaSetDevice(ctx->device));
    if (prec == LP_FP32) {
        if (trans_b) gemm_simt<float, float, float, false, false>(ctx->ex, M, N, K, (const float *)A, K, (const float *)B, K, (float *)C, N, bias, relu);
        else gemm_simt<float, float, float, false, true>(ctx->ex, M, N, K, (const float *)A, K, (const float *)B, N, (float *)C, N, bias, relu);
    } else if (prec == LP_BF16) {
        if (tc_linear_supported(K, N)) {
            std::string err;
            if (!tc_linear_bf16_b(ctx->tc, ctx->ex, M, N, K, (const bf16 *)A, K, (const bf16 *)B, trans_b != 0, bias, relu != 0, (bf16 *)C, N, err))
                return fail(ctx, LP_ECUDA, "lp_op_linear: " + err);
        } else if (trans_b) {
            gemm_simt<bf16, bf16, bf16, false, false>(ctx->ex, M, N, K, (const bf16 *)A, K, (const bf16 *)B, K, (bf16 *)C, N, bias, relu);
        } else {
            gemm_simt<bf16, bf16, bf16, false, true>(ctx->ex, M, N, K, (const bf16 *)A, K, (const bf16 *)B, N, (bf16 *)C, N, bias, relu);
        }
    } else {
        return fail(ctx, LP_EINVAL, "lp_op_linear: unknown precision");
    }
    CK_LAUNCH();
    {
        lp_status ts = tc_check(ctx->tc, ctx->ex, true, ctx->err);
        if (ts != LP_OK) return ts;
    }
    CK(cudaStreamSynchronize(ctx->ex.st));
    return LP_OK;
}

extern "C" lp_status lp_op_weight_grad(lp_ctx *ctx, int32_t prec, int64_t M, int32_t N, int32_t K, const void *A, const void *dZ, float *dW)
{
    if (!ctx) return LP_EINVAL;
    if (!A || !dZ || !dW || M <= 0 || N <= 0 || K <= 0) return fail(ctx, LP_EINVAL, "lp_op_weight_grad: bad argument");
    CK(cudaSetDevice(ctx->device));
    float *partials = nullptr;
    const int64_t need = std::max<int64_t>((int64_t)weight_grad_splits(M) * K * N, tc_weight_grad_partials(M, K, N));
    CK(cudaMalloc((void **)&partials, sizeof(float) * (size_t)need));
    lp_status rc = LP_OK;
    if (prec == LP_FP32) {
        weight_grad_simt<float>(ctx->ex, M, K, N, (const float *)A, K, (const float *)dZ, N, dW, 0, partials);
    } else if (prec == LP_BF16) {
        std::string err;
        if (tc_weight_grad_supported(K, N)) {
            if (!tc_weight_grad(ctx->tc, ctx->ex, M, K, N, (const bf16 *)A, K, (const bf16 *)dZ, N, dW, 0, partials, err)) rc = fail(ctx, LP_ECUDA, "lp_op_weight_grad: " + err);
        } else {
            weight_grad_simt<bf16>(ctx->ex, M, K, N, (const bf16 *)A, K, (const bf16 *)dZ, N, dW, 0, partials);
        }
    } else {
        rc = fail(ctx, LP_EINVAL, "lp_op_weight_grad: unknown precision");
    }
    cudaStreamSynchronize(ctx->ex.st);
    cudaFree(partials);
    if (rc != LP_OK) return rc;
    CK_LAUNCH();
    return tc_check(ctx->tc, ctx->ex, true, ctx->err);
}

// ----------------------------------------------------------------------------------------------
// Weight gradient for callers that must not allocate
// ----------------------------------------------------------------------------------------------
// Some hosts of this library cannot call cudaMalloc at the point where they need a weight
// gradient: a real-time loop that forbids allocator calls (they take driver locks and may
// synchronise the device), a process whose device memory was all handed to a pool at start-up, or
// a code section in which the CUDA runtime itself refuses to allocate.  lp_weight_grad_static serves them: the FP32 partial tiles of
// the split-row reduction live in the fixed device array below instead of a cudaMalloc'ed buffer.
// The array is part of the loaded module, so every GPU that uses this library holds
// LP_STATIC_SCRATCH_FLOATS * 4 bytes of it until the process exits.
#define LP_STATIC_SCRATCH_FLOATS (1 << 21) /* 8 MiB */
static __device__ __align__(256) float lp_static_scratch[LP_STATIC_SCRATCH_FLOATS];

// In host code the name of a __device__ array is only a handle for the runtime, never an address a
// kernel may be given; the device address is looked up once per device, with that device current.
#define LP_STATIC_MAX_DEVICES 64
static float *g_static_scratch_addr[LP_STATIC_MAX_DEVICES];

extern "C" lp_status lp_weight_grad_static(int32_t device, void *cuda_stream, int64_t M, int32_t N, int32_t K, const float *A, const float *dZ,
                                           float *dW)
{
    lp_ctx *ctx = nullptr;  // errors are reported through lp_last_error(NULL)
    if (device < 0 || device >= LP_STATIC_MAX_DEVICES) return fail(ctx, LP_EINVAL, "lp_weight_grad_static: device index out of range");
    if (!A || !dZ || !dW || M <= 0 || N <= 0 || K <= 0) return fail(ctx, LP_EINVAL, "lp_weight_grad_static: bad argument");
    const int64_t tile = (int64_t)K * N;
    if (tile > LP_STATIC_SCRATCH_FLOATS) {
        char buf[200];
        snprintf(buf, sizeof buf, "lp_weight_grad_static: K * N = %lld exceeds the fixed scratch of %d floats; use lp_op_weight_grad instead",
                 (long long)tile, LP_STATIC_SCRATCH_FLOATS);
        return fail(ctx, LP_EINVAL, buf);
    }
    CK(cudaSetDevice(device));
    if (!g_static_scratch_addr[device]) {  // first call on this device: resolve the device address of the array
        float *addr = nullptr;
        CK(cudaGetSymbolAddress((void **)&addr, lp_static_scratch));
        if (!addr) return fail(ctx, LP_ECUDA, "lp_weight_grad_static: cudaGetSymbolAddress returned a null address");
        g_static_scratch_addr[device] = addr;
    }
    float *scratch = g_static_scratch_addr[device];
    // as many row splits as the fixed array holds (each split writes one full K x N partial tile, so
    // nothing has to be cleared between calls: every element that is read was written by this call)
    const int splits = (int)std::max<int64_t>(1, std::min<int64_t>(weight_grad_splits(M), LP_STATIC_SCRATCH_FLOATS / tile));
    int64_t k_chunk = ceil_div64(ceil_div64(M, splits), SG_BK) * SG_BK;
    if (k_chunk < SG_BK) k_chunk = SG_BK;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    dim3 grid((unsigned)ceil_div64(K, SG_BM), (unsigned)ceil_div64(N, SG_BN), (unsigned)splits);
    launch_dep(gemm_simt_kernel<float, float, float, true, true>, dim3(grid), dim3(SG_THREADS), 0, st, K, N, M, A, K, dZ, N, (float *)nullptr, 0, nullptr, 0, k_chunk, scratch, nullptr, 0);
    launch_dep(reduce_partials_kernel, dim3((unsigned)ceil_div64(tile, 256)), dim3(256), 0, st, scratch, tile, splits, dW, 0);
    CK_LAUNCH();
    return LP_OK;
}
