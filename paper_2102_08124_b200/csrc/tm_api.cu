// C ABI of the transposable N:M mask search (see include/tm.h): argument validation, work
// partitioning and kernel dispatch.  Nothing here computes masks on the host.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/tm.h"
#include "tm_launch.h"

namespace {

using tmask::DevProblem;

constexpr int kPartialSlots = 8192;   // objective partials per matrix: (CTAs x warps) of any kernel stays below this
constexpr int kMaxDevices = 64;
constexpr size_t kAlign = 256;
constexpr size_t kHeaderBytes = 256;  // reserved head of every workspace
// Inside the header: the count of finished CTAs of a bandwidth launch that reduces its own objectives.  It is zero
// between launches: cleared once where the library owns the workspace, at the start of the call where the caller does
// (every such launch leaves it at zero again).
constexpr size_t kDoneOffset = 128;
// tm_find_mask_host(): row strips whose copy-in, search and copy-out overlap, and the head of its device workspace (status word,
// then one objective per strip from byte 64 on)
constexpr int kHostStrips = 16;       // 32 and 64 strips measured the same (27.3 ms on a 12288 x 49152 bf16 matrix) and slower (28.4 ms): the bus is the bound
constexpr size_t kHostHead = (64 + 8 * (size_t)kHostStrips + kAlign - 1) / kAlign * kAlign;

size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }
int at_least_one(int count) { return count > 0 ? count : 1; }
size_t table_bytes(int count) { return align_up(sizeof(DevProblem) * (size_t)at_least_one(count)); }
size_t entry_bytes(int count) { return align_up(tmask::tma_entry_bytes() * (size_t)at_least_one(count)); }
size_t partial_bytes(int count) { return align_up(sizeof(double) * (size_t)at_least_one(count) * kPartialSlots); }

// `ready` and `scratch` are published with release stores after the fields they guard are written (under the mutex)
// and read with acquire loads outside it.
struct DeviceState {
    std::atomic<bool> ready{false};
    int sms = 0;
    std::atomic<void*> scratch{nullptr};   // workspace of the plain calls: [status | table | partials]
    size_t scratch_bytes = 0;
    // staging of tm_find_mask_host
    void* stage_w = nullptr; void* stage_masked = nullptr; void* stage_mask = nullptr; void* stage_ws = nullptr; double* stage_obj = nullptr;
    size_t stage_w_bytes = 0, stage_masked_bytes = 0, stage_mask_bytes = 0, stage_ws_bytes = 0;
    cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;

int current_device(DeviceState** st) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return TM_ERR_CUDA; }
    DeviceState& d = g_dev[dev];
    if (!d.ready.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!d.ready.load(std::memory_order_relaxed)) {
            if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
            d.ready.store(true, std::memory_order_release);
        }
    }
    *st = &d;
    return TM_OK;
}

int check_nm(int N, int M) {
    const bool ok = (M == 4 && (N == 1 || N == 2 || N == 3)) || (M == 8 && (N == 2 || N == 4 || N == 6));
    return ok ? TM_OK : TM_ERR_NM;
}
int check_method(int m) { return (m == TM_EXACT || m == TM_APPROX || m == TM_APPROX_COVER) ? TM_OK : TM_ERR_METHOD; }

int check_problem(const tm_problem& p, int M) {
    if (p.dtype != TM_F32 && p.dtype != TM_BF16) return TM_ERR_DTYPE;
    if (p.rows < 0 || p.cols < 0 || p.rows % M || p.cols % M || p.ld < p.cols) return TM_ERR_SHAPE;
    if (p.rows == 0 || p.cols == 0) return TM_OK;
    if (!p.W || !p.mask_out) return TM_ERR_NULL;
    const size_t elem = p.dtype == TM_F32 ? 4 : 2;
    const size_t vec = (size_t)M * elem < 16 ? (size_t)M * elem : 16;    // width of the vector accesses
    if ((uintptr_t)p.W % vec || ((size_t)p.ld * elem) % vec) return TM_ERR_ALIGN;
    if (p.masked_w_out && (uintptr_t)p.masked_w_out % vec) return TM_ERR_ALIGN;
    if ((uintptr_t)p.mask_out % 4 || (p.objective_out && (uintptr_t)p.objective_out % 8)) return TM_ERR_ALIGN;
    return TM_OK;
}

DevProblem to_dev(const tm_problem& p, int M, long long item_begin) {
    DevProblem d;
    d.W = p.W; d.mask = p.mask_out; d.masked = p.masked_w_out; d.objective = p.objective_out;
    d.rows = p.rows; d.cols = p.cols; d.ld = p.ld; d.item_begin = item_begin; d.dtype = p.dtype;
    d.wpr = (int)((p.cols + 31) / 32);
    d.bcols = (int)(p.cols / M);
    d.chunks = (d.bcols + 31) / 32;
    return d;
}

long long items_of(const DevProblem& d, int M) { return (d.rows / M) * (long long)d.chunks; }

// A validated call, partitioned between the bandwidth path and the generic path, with every launch
// argument worked out.  ws layout: [header | table | tma records | partials].
struct PlanGroup {
    bool tma = false;
    int n = 0, used = 0;                     // matrices of the group, offset of the group in every workspace array
    std::vector<DevProblem> probs;           // generic path: the device table's host image
    std::vector<char> entry_store;           // bandwidth path: descriptor records (128-byte aligned inside)
    char* entries = nullptr;
    tmask::LaunchArgs generic;
    tmask::TmaLaunch bandwidth;
};
struct Plan {
    int device = -1, N = 0, M = 0, method = 0, count = 0;
    void* ws = nullptr;
    std::vector<PlanGroup> groups;
};

int validate_call(const tm_problem* probs, int count, int N, int M, int method, void* ws, size_t ws_bytes) {
    int rc;
    if ((rc = check_nm(N, M)) != TM_OK) return rc;
    if ((rc = check_method(method)) != TM_OK) return rc;
    if (count < 0) return TM_ERR_SHAPE;
    if (count == 0) return TM_OK;
    if (!probs) return TM_ERR_NULL;
    for (int k = 0; k < count; ++k)
        if ((rc = check_problem(probs[k], M)) != TM_OK) return rc;
    if (!ws || (uintptr_t)ws % kAlign || ws_bytes < tm_workspace_bytes(probs, count)) return TM_ERR_WORKSPACE;
    return TM_OK;
}

// header_clear: the count of finished CTAs in the workspace's header is zero when the launches start (cleared by this
// library, which also keeps it so), so the bandwidth launches may reduce their own objectives.
int build_plan(const tm_problem* probs, int count, int N, int M, int method, void* ws, size_t ws_bytes, const DeviceState& dev, Plan& plan,
               bool header_clear) {
    const int rc = validate_call(probs, count, N, M, method, ws, ws_bytes);
    if (rc != TM_OK) return rc;
    plan.N = N; plan.M = M; plan.method = method; plan.count = count; plan.ws = ws;
    if (count == 0) return TM_OK;

    char* base = static_cast<char*>(ws);
    DevProblem* dtab = reinterpret_cast<DevProblem*>(base + kHeaderBytes);
    char* dent = base + kHeaderBytes + table_bytes(count);
    double* dpart = reinterpret_cast<double*>(dent + entry_bytes(count));

    // group 0: generic; groups 1..4: bandwidth path by (dtype, masked output present)
    std::vector<DevProblem> group[5];
    // A lane of the staged kernel scores its four blocks of an item one after the other: a small exact call is spread
    // wider, and finished sooner, by the generic kernel (one block per lane).
    long long call_weights = 0;
    for (int k = 0; k < count; ++k) call_weights += (long long)probs[k].rows * probs[k].cols;
    const bool staged = !(method == TM_EXACT && call_weights < (1ll << 20));
    for (int k = 0; k < count; ++k) {
        DevProblem d = to_dev(probs[k], M, 0);
        const int g = staged && tmask::tma_eligible(d, N, M, method) ? 1 + 2 * d.dtype + (d.masked ? 1 : 0) : 0;
        group[g].push_back(d);
    }
    int used = 0;
    for (int g = 0; g < 5; ++g) {
        const int n = (int)group[g].size();
        if (n == 0) continue;
        plan.groups.emplace_back();
        PlanGroup& pg = plan.groups.back();
        pg.tma = g != 0; pg.n = n; pg.used = used;
        double* partials = dpart + (size_t)used * kPartialSlots;
        if (g == 0) {
            pg.probs = group[g];
            long long total = 0;
            for (int k = 0; k < n; ++k) { pg.probs[k].item_begin = total; total += items_of(pg.probs[k], M); }
            tmask::LaunchArgs& a = pg.generic;
            a.count = n; a.total_items = total; a.N = N; a.M = M; a.method = method; a.stream = nullptr; a.status = nullptr;
            a.partials = partials;
            const int wpc = tmask::generic_warps_per_cta(N, M, method);
            const long long want = (total + wpc - 1) / wpc;
            const int fill = dev.sms * tmask::generic_ctas_per_sm(N, M, method);
            const int cap = fill < kPartialSlots / wpc ? fill : kPartialSlots / wpc;
            a.ctas = (int)(want < 1 ? 1 : (want > cap ? cap : want));
            a.single = pg.probs[0];
            a.table = n > 1 ? dtab + used : nullptr;
        } else {
            const size_t esz = tmask::tma_entry_bytes();
            pg.entry_store.resize(esz * (size_t)n + 128);
            pg.entries = pg.entry_store.data() + ((128 - (uintptr_t)pg.entry_store.data() % 128) % 128);
            long long total = 0;
            if (!tmask::tma_build_entries(group[g].data(), n, pg.entries, &total, M, method)) return TM_ERR_CUDA;
            tmask::TmaLaunch& a = pg.bandwidth;
            a.entries_host = pg.entries; a.count = n; a.total_items = total; a.partials = partials;
            a.status = nullptr; a.dtype = (g - 1) / 2; a.method = method; a.M = M; a.has_out = ((g - 1) & 1) != 0; a.stream = nullptr;
            const int wpc = tmask::tma_warps_per_cta(a.dtype, M, method);
            const long long want = (total + wpc - 1) / wpc;
            const int cap = dev.sms < kPartialSlots / wpc ? dev.sms : kPartialSlots / wpc;
            a.ctas = (int)(want < 1 ? 1 : (want > cap ? cap : want));
            a.entries_dev = n > 1 ? dent + (size_t)used * esz : nullptr;
            a.done = header_clear ? reinterpret_cast<unsigned int*>(base + kDoneOffset) : nullptr;
        }
        used += n;
    }
    return TM_OK;
}

// Copies the descriptor tables of multi-matrix groups into the workspace (pageable sources: the runtime
// stages the bytes before cudaMemcpyAsync returns -- waiting for the stream's earlier work if it has to -- so the
// plan may die right after).  Such a copy cannot be recorded by a stream capture (a replay would read host memory
// that is long gone): a call that needs one while its stream is capturing is refused.
int upload_plan(const Plan& plan, cudaStream_t stream) {
    bool needed = false;
    for (const PlanGroup& pg : plan.groups) needed |= pg.n > 1;
    if (!needed) return TM_OK;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    if (cap != cudaStreamCaptureStatusNone) return TM_ERR_CAPTURE;
    for (const PlanGroup& pg : plan.groups) {
        if (pg.n <= 1) continue;
        cudaError_t e = pg.tma
            ? cudaMemcpyAsync(const_cast<void*>(pg.bandwidth.entries_dev), pg.entries, tmask::tma_entry_bytes() * (size_t)pg.n, cudaMemcpyHostToDevice, stream)
            : cudaMemcpyAsync(const_cast<DevProblem*>(pg.generic.table), pg.probs.data(), sizeof(DevProblem) * (size_t)pg.n, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    }
    return TM_OK;
}

// Kernel launches (and the clearing of their partials) only: nothing here touches host memory asynchronously.
int launch_plan(const Plan& plan, int* status_dev, cudaStream_t stream) {
    for (const PlanGroup& pg : plan.groups) {
        cudaError_t e;
        if (pg.tma) { tmask::TmaLaunch a = pg.bandwidth; a.status = status_dev; a.stream = stream; e = tmask::launch_tma(a); }
        else { tmask::LaunchArgs a = pg.generic; a.status = status_dev; a.stream = stream; e = tmask::launch_generic(a); }
        if (e != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    }
    return TM_OK;
}

// What is known of the workspace's header when a call starts: cleared by this library and untouched since; contents
// unknown (the count of finished CTAs is cleared on the stream first -- four bytes instead of the objective partials, and no
// reduction kernel); or left alone (the launches clear their partials and a reduction kernel follows them).
enum HeaderState { kHeaderClear, kHeaderUnknown, kHeaderUnused };

int run(const tm_problem* probs, int count, int N, int M, int method, void* ws, size_t ws_bytes, int* status_dev,
        cudaStream_t stream, const DeviceState& dev, HeaderState header) {
    Plan plan;
    int rc = build_plan(probs, count, N, M, method, ws, ws_bytes, dev, plan, header != kHeaderUnused);
    if (rc != TM_OK) return rc;
    if ((rc = upload_plan(plan, stream)) != TM_OK) return rc;
    if (header == kHeaderUnknown) {
        bool wanted = false;
        for (const PlanGroup& pg : plan.groups) wanted |= pg.tma && pg.bandwidth.done != nullptr;
        if (wanted && cudaMemsetAsync(static_cast<char*>(ws) + kDoneOffset, 0, sizeof(unsigned int), stream) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    }
    return launch_plan(plan, status_dev, stream);
}

int ensure_scratch(DeviceState& d) {
    if (d.scratch.load(std::memory_order_acquire)) return TM_OK;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (d.scratch.load(std::memory_order_relaxed)) return TM_OK;
    const size_t bytes = tm_workspace_bytes(nullptr, 1);
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    if (cudaMemset(p, 0, kHeaderBytes) != cudaSuccess) { cudaGetLastError(); cudaFree(p); return TM_ERR_CUDA; }
    d.scratch_bytes = bytes;
    d.scratch.store(p, std::memory_order_release);
    return TM_OK;
}

int plain_call(const void* W, int dtype, int64_t rows, int64_t cols, int N, int M, int method,
               uint32_t* mask_out, void* masked_w_out, double* objective_out) {
    tm_problem p;
    p.W = W; p.rows = rows; p.cols = cols; p.ld = cols; p.dtype = dtype;
    p.mask_out = mask_out; p.masked_w_out = masked_w_out; p.objective_out = objective_out;
    // validate before touching the device
    int rc;
    if ((rc = check_nm(N, M)) != TM_OK) return rc;
    if ((rc = check_method(method)) != TM_OK) return rc;
    if ((rc = check_problem(p, M)) != TM_OK) return rc;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != TM_OK) return rc;
    if ((rc = ensure_scratch(*d)) != TM_OK) return rc;
    void* scratch = d->scratch.load(std::memory_order_acquire);
    return run(&p, 1, N, M, method, scratch, d->scratch_bytes, static_cast<int*>(scratch), nullptr, *d, kHeaderClear);
}

int grow(void** p, size_t* have, size_t want) {
    if (*have >= want) return TM_OK;
    if (*p) cudaFree(*p);
    *p = nullptr; *have = 0;
    if (cudaMalloc(p, want) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    *have = want;
    return TM_OK;
}

// ---- built-in scratch of tm_find_mask_batched_static() ------------------------------------------
// In host code the array's name is only a handle for the runtime, not a device address: the
// address the kernels may use comes from cudaGetSymbolAddress(), looked up once per device.
static __device__ __align__(256) unsigned char g_static_scratch[TM_STATIC_SCRATCH_BYTES];

struct StaticScratch {
    std::atomic<void*> ptr{nullptr};       // published once the look-up has succeeded
};
StaticScratch g_static[kMaxDevices];

int static_scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return TM_ERR_CUDA; }
    StaticScratch& s = g_static[dev];
    void* p = s.ptr.load(std::memory_order_acquire);
    if (!p) {
        std::lock_guard<std::mutex> lock(g_mutex);
        p = s.ptr.load(std::memory_order_relaxed);
        if (!p) {
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return TM_ERR_CUDA; }
            s.ptr.store(p, std::memory_order_release);
        }
    }
    *out = p;
    return TM_OK;
}

}  // namespace

extern "C" {

size_t tm_mask_words_per_row(int64_t cols) { return cols > 0 ? (size_t)((cols + 31) / 32) : 0; }
size_t tm_mask_words(int64_t rows, int64_t cols) { return rows > 0 ? (size_t)rows * tm_mask_words_per_row(cols) : 0; }

size_t tm_workspace_bytes(const tm_problem* /*probs_host*/, int count) {
    return kHeaderBytes + table_bytes(count) + entry_bytes(count) + partial_bytes(count);
}

int tm_find_mask(const void* W, int64_t rows, int64_t cols, int N, int M, int method,
                 uint32_t* mask_out, void* masked_w_out, double* objective_out) {
    return plain_call(W, TM_F32, rows, cols, N, M, method, mask_out, masked_w_out, objective_out);
}

int tm_find_mask_bf16(const void* W, int64_t rows, int64_t cols, int N, int M, int method,
                      uint32_t* mask_out, void* masked_w_out, double* objective_out) {
    return plain_call(W, TM_BF16, rows, cols, N, M, method, mask_out, masked_w_out, objective_out);
}

int tm_device_status(int* status_host) {
    if (!status_host) return TM_ERR_NULL;
    DeviceState* d = nullptr;
    int rc = current_device(&d);
    if (rc != TM_OK) return rc;
    *status_host = 0;
    void* scratch = d->scratch.load(std::memory_order_acquire);
    if (!scratch) return TM_OK;
    if (cudaStreamSynchronize(nullptr) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    if (cudaMemcpy(status_host, scratch, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    if (cudaMemset(scratch, 0, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    return TM_OK;
}

int tm_find_mask_batched(const tm_problem* probs_host, int count, int N, int M, int method,
                         void* workspace_dev, size_t workspace_bytes, int* status_dev, void* cuda_stream) {
    int rc;
    if ((rc = check_nm(N, M)) != TM_OK) return rc;
    if ((rc = check_method(method)) != TM_OK) return rc;
    if (count < 0) return TM_ERR_SHAPE;
    if (count > 0 && !probs_host) return TM_ERR_NULL;
    for (int k = 0; k < count; ++k)
        if ((rc = check_problem(probs_host[k], M)) != TM_OK) return rc;
    if (count > 0 && (!workspace_dev || (uintptr_t)workspace_dev % kAlign || workspace_bytes < tm_workspace_bytes(probs_host, count)))
        return TM_ERR_WORKSPACE;
    if (count == 0) return TM_OK;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != TM_OK) return rc;
    return run(probs_host, count, N, M, method, workspace_dev, workspace_bytes, status_dev, static_cast<cudaStream_t>(cuda_stream), *d, kHeaderUnknown);
}

int tm_find_mask_host(const void* W_host, int dtype, int64_t rows, int64_t cols, int N, int M, int method,
                      uint32_t* mask_out_host, void* masked_w_out_host, double* objective_out_host, int* status_out_host) {
    int rc;
    if ((rc = check_nm(N, M)) != TM_OK) return rc;
    if ((rc = check_method(method)) != TM_OK) return rc;
    if (dtype != TM_F32 && dtype != TM_BF16) return TM_ERR_DTYPE;
    if (rows < 0 || cols < 0 || rows % M || cols % M) return TM_ERR_SHAPE;
    if (status_out_host) *status_out_host = 0;
    if (objective_out_host) *objective_out_host = 0.0;
    if (rows == 0 || cols == 0) return TM_OK;
    if (!W_host || !mask_out_host) return TM_ERR_NULL;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != TM_OK) return rc;

    const size_t elem = dtype == TM_F32 ? 4 : 2;
    const size_t row_bytes = (size_t)cols * elem, wpr = tm_mask_words_per_row(cols);
    // row strips: copy-in, search and copy-out of neighbouring strips overlap on three streams
    const int64_t brows = rows / M;
    const int strips = (int)(brows < kHostStrips ? brows : kHostStrips);
    const int64_t strip_brows = (brows + strips - 1) / strips;
    const size_t one_ws = tm_workspace_bytes(nullptr, 1);
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!d->s_in) {
            if (cudaStreamCreateWithFlags(&d->s_in, cudaStreamNonBlocking) != cudaSuccess ||
                cudaStreamCreateWithFlags(&d->s_run, cudaStreamNonBlocking) != cudaSuccess ||
                cudaStreamCreateWithFlags(&d->s_out, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
        }
        if ((rc = grow(&d->stage_w, &d->stage_w_bytes, (size_t)rows * row_bytes)) != TM_OK) return rc;
        if (masked_w_out_host && (rc = grow(&d->stage_masked, &d->stage_masked_bytes, (size_t)rows * row_bytes)) != TM_OK) return rc;
        if ((rc = grow(&d->stage_mask, &d->stage_mask_bytes, (size_t)rows * wpr * 4)) != TM_OK) return rc;
        if ((rc = grow(&d->stage_ws, &d->stage_ws_bytes, (one_ws + kAlign) * kHostStrips + kHostHead)) != TM_OK) return rc;
    }
    char* ws = static_cast<char*>(d->stage_ws);
    int* status_dev = reinterpret_cast<int*>(ws);                       // the head: status, then the strips' objectives
    double* obj_dev = reinterpret_cast<double*>(ws + 64);
    // status and objectives, and the headers of the strips' workspaces (their launches count finished CTAs there)
    if (cudaMemsetAsync(ws, 0, (one_ws + kAlign) * kHostStrips + kHostHead, d->s_run) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }

    std::vector<cudaEvent_t> ev_in((size_t)strips), ev_run((size_t)strips);
    bool ok = true;
    for (int s = 0; s < strips && ok; ++s) {
        ok &= cudaEventCreateWithFlags(&ev_in[s], cudaEventDisableTiming) == cudaSuccess;
        ok &= cudaEventCreateWithFlags(&ev_run[s], cudaEventDisableTiming) == cudaSuccess;
    }
    for (int s = 0; s < strips && ok; ++s) {
        const int64_t r0 = s * strip_brows * M;
        int64_t r1 = (s + 1) * strip_brows * M; if (r1 > rows) r1 = rows;
        if (r0 >= r1) { ok &= cudaEventRecord(ev_in[s], d->s_in) == cudaSuccess; ok &= cudaEventRecord(ev_run[s], d->s_run) == cudaSuccess; continue; }
        const size_t off = (size_t)r0 * row_bytes, nbytes = (size_t)(r1 - r0) * row_bytes;
        ok &= cudaMemcpyAsync(static_cast<char*>(d->stage_w) + off, static_cast<const char*>(W_host) + off, nbytes, cudaMemcpyHostToDevice, d->s_in) == cudaSuccess;
        ok &= cudaEventRecord(ev_in[s], d->s_in) == cudaSuccess;
        ok &= cudaStreamWaitEvent(d->s_run, ev_in[s], 0) == cudaSuccess;
        tm_problem p;
        p.W = static_cast<char*>(d->stage_w) + off; p.rows = r1 - r0; p.cols = cols; p.ld = cols; p.dtype = dtype;
        p.mask_out = static_cast<uint32_t*>(d->stage_mask) + (size_t)r0 * wpr;
        p.masked_w_out = masked_w_out_host ? static_cast<char*>(d->stage_masked) + off : nullptr;
        p.objective_out = obj_dev + s;
        rc = run(&p, 1, N, M, method, ws + kHostHead + (size_t)s * (one_ws + kAlign), one_ws, status_dev, d->s_run, *d, kHeaderClear);
        if (rc != TM_OK) { ok = false; break; }
        ok &= cudaEventRecord(ev_run[s], d->s_run) == cudaSuccess;
        ok &= cudaStreamWaitEvent(d->s_out, ev_run[s], 0) == cudaSuccess;
        ok &= cudaMemcpyAsync(mask_out_host + (size_t)r0 * wpr, p.mask_out, (size_t)(r1 - r0) * wpr * 4, cudaMemcpyDeviceToHost, d->s_out) == cudaSuccess;
        if (masked_w_out_host)
            ok &= cudaMemcpyAsync(static_cast<char*>(masked_w_out_host) + off, p.masked_w_out, nbytes, cudaMemcpyDeviceToHost, d->s_out) == cudaSuccess;
    }
    double obj_host[kHostStrips] = {0}; int status_host = 0;
    if (ok) {
        ok &= cudaStreamSynchronize(d->s_run) == cudaSuccess;
        ok &= cudaMemcpy(obj_host, obj_dev, sizeof(double) * (size_t)strips, cudaMemcpyDeviceToHost) == cudaSuccess;
        ok &= cudaMemcpy(&status_host, status_dev, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess;
        ok &= cudaStreamSynchronize(d->s_out) == cudaSuccess;
    } else {
        cudaStreamSynchronize(d->s_in); cudaStreamSynchronize(d->s_run); cudaStreamSynchronize(d->s_out);
    }
    for (int s = 0; s < strips; ++s) { if (ev_in[s]) cudaEventDestroy(ev_in[s]); if (ev_run[s]) cudaEventDestroy(ev_run[s]); }
    if (!ok) { cudaGetLastError(); return rc != TM_OK ? rc : TM_ERR_CUDA; }
    if (objective_out_host) { double t = 0.0; for (int s = 0; s < strips; ++s) t += obj_host[s]; *objective_out_host = t; }
    if (status_out_host) *status_out_host = status_host;
    return TM_OK;
}

int tm_find_mask_batched_static(const tm_problem* probs_host, int count, int N, int M, int method,
                                int* status_dev, void* cuda_stream) {
    int rc;
    if ((rc = check_nm(N, M)) != TM_OK) return rc;
    if ((rc = check_method(method)) != TM_OK) return rc;
    if (count < 0) return TM_ERR_SHAPE;
    if (count > TM_STATIC_MAX_MATRICES) return TM_ERR_TOO_LARGE;
    if (count > 0 && !probs_host) return TM_ERR_NULL;
    for (int k = 0; k < count; ++k)
        if ((rc = check_problem(probs_host[k], M)) != TM_OK) return rc;
    if (count == 0) return TM_OK;
    if (tm_workspace_bytes(probs_host, TM_STATIC_MAX_MATRICES) > (size_t)TM_STATIC_SCRATCH_BYTES) return TM_ERR_WORKSPACE;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != TM_OK) return rc;
    void* scratch = nullptr;
    if ((rc = static_scratch_address(&scratch)) != TM_OK) return rc;
    // every launch below clears the objective partials it uses before its kernel runs on the same stream
    return run(probs_host, count, N, M, method, scratch, TM_STATIC_SCRATCH_BYTES, status_dev, static_cast<cudaStream_t>(cuda_stream), *d, kHeaderUnused);
}

struct tm_plan { Plan plan; };

int tm_plan_create(const tm_problem* probs_host, int count, int N, int M, int method, void* workspace_dev, size_t workspace_bytes,
                   tm_plan** plan_out) {
    if (!plan_out) return TM_ERR_NULL;
    *plan_out = nullptr;
    DeviceState* d = nullptr;
    int rc;
    // validate before touching the device
    if ((rc = validate_call(probs_host, count, N, M, method, workspace_dev, workspace_bytes)) != TM_OK) return rc;
    if ((rc = current_device(&d)) != TM_OK) return rc;
    tm_plan* p = new (std::nothrow) tm_plan();
    if (!p) return TM_ERR_CUDA;
    // the plan owns the workspace from here on: its header is cleared once, below, and single-matrix launches keep it clear
    if ((rc = build_plan(probs_host, count, N, M, method, workspace_dev, workspace_bytes, *d, p->plan, true)) != TM_OK) { delete p; return rc; }
    if (count > 0 && cudaMemset(workspace_dev, 0, kHeaderBytes) != cudaSuccess) { cudaGetLastError(); delete p; return TM_ERR_CUDA; }
    cudaGetDevice(&p->plan.device);
    // the tables are uploaded once, synchronously: tm_plan_run() then issues kernels only
    if ((rc = upload_plan(p->plan, nullptr)) != TM_OK || cudaStreamSynchronize(nullptr) != cudaSuccess) { cudaGetLastError(); delete p; return rc != TM_OK ? rc : TM_ERR_CUDA; }
    *plan_out = p;
    return TM_OK;
}

int tm_plan_run(const tm_plan* plan, int* status_dev, void* cuda_stream) {
    if (!plan) return TM_ERR_NULL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != plan->plan.device) { cudaGetLastError(); return TM_ERR_CUDA; }
    return launch_plan(plan->plan, status_dev, static_cast<cudaStream_t>(cuda_stream));
}

void tm_plan_destroy(tm_plan* plan) { delete plan; }

size_t tm_aux_workspace_bytes(void) { return kHeaderBytes + 2 * sizeof(double) * (size_t)tmask::aux_partial_slots(); }

namespace {
int check_aux_matrix(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, int M) {
    if (dtype != TM_F32 && dtype != TM_BF16) return TM_ERR_DTYPE;
    if (rows < 0 || cols < 0 || cols % M || ld < cols) return TM_ERR_SHAPE;
    if (rows == 0 || cols == 0) return TM_OK;
    if (!W) return TM_ERR_NULL;
    const size_t elem = dtype == TM_F32 ? 4 : 2;
    const size_t vec = (size_t)M * elem < 16 ? (size_t)M * elem : 16;
    if ((uintptr_t)W % vec || ((size_t)ld * elem) % vec) return TM_ERR_ALIGN;
    return TM_OK;
}
int check_aux_workspace(void* ws, size_t bytes) {
    return (!ws || (uintptr_t)ws % kAlign || bytes < tm_aux_workspace_bytes()) ? TM_ERR_WORKSPACE : TM_OK;
}
}  // namespace

int tm_nm_mask_1d(const tm_problem* prob_host, int N, int M, int flags, unsigned long long* violations_out,
                  void* workspace_dev, size_t workspace_bytes, int* status_dev, void* cuda_stream) {
    if (!prob_host) return TM_ERR_NULL;
    if ((M != 2 && M != 4 && M != 8) || N < 0 || N > M) return TM_ERR_NM;
    const tm_problem& p = *prob_host;
    int rc;
    if ((rc = check_aux_matrix(p.W, p.dtype, p.rows, p.cols, p.ld, M)) != TM_OK) return rc;
    if (p.rows > 0 && p.cols > 0) {
        if (!p.mask_out) return TM_ERR_NULL;
        const size_t elem = p.dtype == TM_F32 ? 4 : 2, vec = (size_t)M * elem < 16 ? (size_t)M * elem : 16;
        if ((uintptr_t)p.mask_out % 4 || (p.masked_w_out && (uintptr_t)p.masked_w_out % vec) || (p.objective_out && (uintptr_t)p.objective_out % 8) ||
            (violations_out && (uintptr_t)violations_out % 8)) return TM_ERR_ALIGN;
    }
    if ((rc = check_aux_workspace(workspace_dev, workspace_bytes)) != TM_OK) return rc;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != TM_OK) return rc;
    tmask::AuxProblem a;
    a.W = p.W; a.mask = p.mask_out; a.masked = p.masked_w_out; a.rows = p.rows; a.cols = p.cols; a.ld = p.ld; a.dtype = p.dtype;
    a.wpr = (int)((p.cols + 31) / 32);
    char* base = static_cast<char*>(workspace_dev) + kHeaderBytes;
    double* op = reinterpret_cast<double*>(base);
    unsigned long long* vp = reinterpret_cast<unsigned long long*>(base + sizeof(double) * (size_t)tmask::aux_partial_slots());
    // groups of four and of eight ride the bandwidth kernels of the searches (row rule instead of steps A-C); the mean
    // absorption only for groups of four
    const bool absorb = (flags & TM_NM1D_ABSORB_MEAN) && p.masked_w_out != nullptr;
    if (((M == 4 && N >= 1 && N <= 3) || (M == 8 && N >= 1 && N <= 7 && !absorb)) && p.rows > 0 && p.cols > 0) {
        const DevProblem dp = to_dev(p, M, 0);
        const int rows_method = absorb ? tmask::kMethodRowsAbsorb : tmask::kMethodRows;
        if (tmask::tma_eligible(dp, N, M, rows_method)) {
            alignas(128) unsigned char entry[512];
            long long total = 0;
            if (tmask::tma_entry_bytes() <= sizeof(entry) && tmask::tma_build_entries(&dp, 1, entry, &total, M, rows_method)) {
                tmask::TmaLaunch t;
                t.entries_host = entry; t.entries_dev = nullptr; t.count = 1; t.total_items = total; t.partials = op; t.status = status_dev;
                t.dtype = p.dtype; t.M = M; t.has_out = p.masked_w_out != nullptr;
                t.method = rows_method;
                t.stream = static_cast<cudaStream_t>(cuda_stream); t.n_keep = N; t.vpartials = vp;
                const int wpc = tmask::tma_warps_per_cta(t.dtype, M, t.method);
                const long long want = (total + wpc - 1) / wpc;
                const int cap = d->sms < tmask::aux_partial_slots() / wpc ? d->sms : tmask::aux_partial_slots() / wpc;
                t.ctas = (int)(want < 1 ? 1 : (want > cap ? cap : want));
                if (tmask::launch_tma(t) != cudaSuccess ||
                    tmask::launch_aux_reduce(op, vp, t.ctas * wpc, p.objective_out, violations_out, t.stream) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
                return TM_OK;
            }
        }
    }
    if (tmask::launch_nm1d(a, N, M, flags, false, op, vp, p.objective_out, violations_out, status_dev, d->sms,
                           static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    return TM_OK;
}

int tm_mask_violations(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, const uint32_t* mask,
                       unsigned long long* violations_out, void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
    int rc;
    if ((rc = check_aux_matrix(W, dtype, rows, cols, ld, 1)) != TM_OK) return rc;
    if (!violations_out || (rows > 0 && cols > 0 && !mask)) return TM_ERR_NULL;
    if ((uintptr_t)mask % 4 || (uintptr_t)violations_out % 8) return TM_ERR_ALIGN;
    if ((rc = check_aux_workspace(workspace_dev, workspace_bytes)) != TM_OK) return rc;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != TM_OK) return rc;
    tmask::AuxProblem a;
    a.W = W; a.mask = const_cast<uint32_t*>(mask); a.masked = nullptr; a.rows = rows; a.cols = cols; a.ld = ld; a.dtype = dtype;
    a.wpr = (int)((cols + 31) / 32);
    char* base = static_cast<char*>(workspace_dev) + kHeaderBytes;
    double* op = reinterpret_cast<double*>(base);
    unsigned long long* vp = reinterpret_cast<unsigned long long*>(base + sizeof(double) * (size_t)tmask::aux_partial_slots());
    if (tmask::launch_nm1d(a, 0, 8, 0, true, op, vp, nullptr, violations_out, nullptr, d->sms,
                           static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) { cudaGetLastError(); return TM_ERR_CUDA; }
    return TM_OK;
}

int tm_mask_hamming(const uint32_t* mask_a, const uint32_t* mask_b, int64_t words, unsigned long long* distance_out,
                    void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
    if (words < 0) return TM_ERR_SHAPE;
    if (!distance_out || (words > 0 && (!mask_a || !mask_b))) return TM_ERR_NULL;
    if ((uintptr_t)mask_a % 4 || (uintptr_t)mask_b % 4 || (uintptr_t)distance_out % 8) return TM_ERR_ALIGN;
    int rc;
    if ((rc = check_aux_workspace(workspace_dev, workspace_bytes)) != TM_OK) return rc;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != TM_OK) return rc;
    unsigned long long* vp = reinterpret_cast<unsigned long long*>(static_cast<char*>(workspace_dev) + kHeaderBytes);
    if (tmask::launch_hamming(mask_a, mask_b, words, vp, distance_out, d->sms, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        cudaGetLastError(); return TM_ERR_CUDA;
    }
    return TM_OK;
}

int tm_compress_2_4(const void* W, int dtype, int64_t rows, int64_t cols, int64_t ld, const uint32_t* mask,
                    void* values, uint32_t* meta, void* values_t, uint32_t* meta_t, int* status_dev, void* cuda_stream) {
    int rc;
    if (rows % 4) return TM_ERR_SHAPE;
    if ((rc = check_aux_matrix(W, dtype, rows, cols, ld, 4)) != TM_OK) return rc;
    if (rows == 0 || cols == 0) return TM_OK;
    if (!mask || !values || !meta || !values_t || !meta_t) return TM_ERR_NULL;
    if ((uintptr_t)mask % 4 || (uintptr_t)meta % 4 || (uintptr_t)meta_t % 4 || (uintptr_t)values % 8 || (uintptr_t)values_t % 4) return TM_ERR_ALIGN;
    DeviceState* d = nullptr;
    if ((rc = current_device(&d)) != TM_OK) return rc;
    tmask::AuxProblem a;
    a.W = W; a.mask = const_cast<uint32_t*>(mask); a.masked = nullptr; a.rows = rows; a.cols = cols; a.ld = ld; a.dtype = dtype;
    a.wpr = (int)((cols + 31) / 32);
    if (tmask::launch_compress24(a, values, meta, values_t, meta_t, status_dev, d->sms, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        cudaGetLastError(); return TM_ERR_CUDA;
    }
    return TM_OK;
}

const char* tm_status_string(int code) {
    switch (code) {
    case TM_OK: return "ok";
    case TM_ERR_NULL: return "a required pointer is NULL";
    case TM_ERR_SHAPE: return "bad shape: sizes must be non-negative multiples of M and ld >= cols";
    case TM_ERR_NM: return "unsupported (N, M)";
    case TM_ERR_METHOD: return "unknown method";
    case TM_ERR_DTYPE: return "unknown dtype";
    case TM_ERR_ALIGN: return "misaligned pointer or row pitch";
    case TM_ERR_CUDA: return "CUDA runtime error (no device, launch or allocation failure)";
    case TM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case TM_ERR_TOO_LARGE: return "too many matrices for the built-in scratch (TM_STATIC_MAX_MATRICES per call)";
    case TM_ERR_CAPTURE: return "the stream is being captured and the call would have to copy descriptor tables from host memory (use tm_plan_run)";
    default: return "unknown status";
    }
}

int tm_version(void) { return TM_VERSION; }

}  // extern "C"
