// Host side of the executor: binds a plan's tables into a workspace, launches the kernels (kernel_*.cu) and
// reads their verdict; also the host pipeline for AllToAllv through host buffers, the resident executor's
// doorbell calls and the no-allocation entry point.
#include "bulk_layout.h"
#include "kernels.cuh"

// ====================================================================== host side
using namespace hccl;

namespace {
thread_local char g_cuda_err[256] = "";
hccl_status_t cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return HCCL_ERR_CUDA;
}
#define CUDA_TRY(x)                                   \
    do {                                              \
        cudaError_t _e = (x);                         \
        if (_e != cudaSuccess) return cuda_fail(_e, #x); \
    } while (0)
}  // namespace

extern "C" {

const char* hccl_last_cuda_error(void) { return g_cuda_err; }

hccl_status_t hccl_plan_bind(hccl_plan_t* p, void* dev_workspace, size_t bytes, void* stream) {
    if (!p || !dev_workspace) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)dev_workspace) % 256) return HCCL_ERR_ALIGNMENT;
    if (bytes < p->layout.total) return HCCL_ERR_WORKSPACE;
    const Layout& L = p->layout;
    std::vector<char> img((size_t)L.scratch, 0);  // control, counters and signals start at zero
    if (!p->descs.empty()) std::memcpy(img.data() + L.descs, p->descs.data(), p->descs.size() * sizeof(Desc));
    if (!p->tiles.empty()) std::memcpy(img.data() + L.tiles, p->tiles.data(), p->tiles.size() * sizeof(Tile));
    if (!p->waits.empty()) std::memcpy(img.data() + L.waits, p->waits.data(), p->waits.size() * sizeof(Wait));
    cudaStream_t s = (cudaStream_t)stream;
    CUDA_TRY(cudaMemcpyAsync(dev_workspace, img.data(), img.size(), cudaMemcpyHostToDevice, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    // opt-in shared memory sizes are set here, once, so that hccl_execute itself is only a launch
    if (p->dynamic && !p->dyn_device_tables) {
        const size_t RR = (size_t)p->R * p->R;
        const size_t smem = RR * 24 + (RR + 1) * 4 + 16;
        if (smem > 48 * 1024) CUDA_TRY(cudaFuncSetAttribute(hccl_a2a_dynamic, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(DYN_MAX_RANKS * DYN_MAX_RANKS * 24 + (DYN_MAX_RANKS * DYN_MAX_RANKS + 1) * 4 + 16)));
    } else if (p->opts.engine == HCCL_ENGINE_BULK) {
        CUDA_TRY(cudaFuncSetAttribute(hccl_executor_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bulk::MAX_DYNAMIC_SMEM));
        if (p->chain_len) {
            CUDA_TRY(cudaFuncSetAttribute(hccl_executor_chain, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CHAIN_SMEM_BYTES));
            CUDA_TRY(cudaFuncSetAttribute(hccl_executor_chain_sums, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CHAIN_SMEM_BYTES));
        }
    }
    p->workspace = dev_workspace;
    p->workspace_bytes = bytes;
    p->epoch = 0;
    p->checked_send.clear();
    p->checked_recv.clear();
    return HCCL_OK;
}

// How the blocks find their work: tickets, one item per block, or static chains.
static int set_dispatch(const hccl_plan_t* p, ExecParams& prm) {
    int blocks = p->opts.sm_budget;
    if ((uint32_t)blocks > prm.n_tiles) blocks = (int)std::max<uint32_t>(prm.n_tiles, 1u);
    prm.chain_len = p->chain_len;
    prm.n_chains = p->n_chains;
    prm.host_completed = nullptr;
    prm.host_t_done = nullptr;
    prm.first_epoch = 0;
    prm.pad2 = 0;
    if (p->chain_len) blocks = (int)std::max<uint32_t>(1u, std::min<uint32_t>((uint32_t)blocks, p->n_chains));
    prm.static_tickets = (!p->chain_len && prm.n_waits == 0 && prm.n_tiles <= (uint32_t)blocks) ? 1 : 0;
    prm.quantum = 0;
    if (p->opts.quantum > 0 && !p->chain_len && !p->dynamic && prm.n_tiles > 0) {
        // short-lived blocks: as many as it takes when each one leaves after `quantum` items; how many run at once
        // is up to the hardware's block scheduler (and to the stream's priority against other work)
        prm.quantum = (uint32_t)p->opts.quantum;
        prm.static_tickets = 0;
        blocks = (int)std::min<uint64_t>(((uint64_t)prm.n_tiles + prm.quantum - 1) / prm.quantum, 1u << 20);
        if ((uint64_t)blocks * prm.quantum < prm.n_tiles) prm.quantum = (uint32_t)(((uint64_t)prm.n_tiles + blocks - 1) / blocks);
    }
    prm.nblocks = (uint32_t)blocks;
    return blocks;
}

// Kernel parameters of a bound plan: table addresses inside its workspace, sizes, trigger, rank buffers, and
// how the blocks find their work. Returns the number of blocks to launch.
static int fill_params(const hccl_plan_t* p, ExecParams& prm, const void* const* sendbufs, void* const* recvbufs) {
    char* ws = (char*)p->workspace;
    const Layout& L = p->layout;
    prm.descs = (const Desc*)(ws + L.descs);
    prm.tiles = (const Tile*)(ws + L.tiles);
    prm.waits = (const Wait*)(ws + L.waits);
    prm.counters = (uint32_t*)(ws + L.counters);
    prm.signals = (unsigned long long*)(ws + L.signals);
    prm.ctl = (Control*)(ws + L.control);
    prm.scratch = ws + L.scratch;
    prm.user_signals = (unsigned long long*)p->user_signals;
    prm.trace = (unsigned long long*)p->trace;
    prm.trace_cap = (unsigned long long)p->trace_cap;
    prm.n_tiles = (uint32_t)p->tiles.size();
    prm.n_descs = (uint32_t)p->descs.size();
    prm.n_syncs = (uint32_t)p->sync_per_epoch.size();
    prm.n_waits = (uint32_t)p->waits.size();
    prm.n_signals = (uint32_t)p->n_signals;
    prm.R = (uint32_t)p->R;
    prm.timeout_ns = p->opts.timeout_ns;
    prm.n_user_signals = p->n_user_signals;
    prm.trig_wait_slot = p->trig_wait_slot;
    prm.trig_set_slot = p->trig_set_slot;
    prm.trig_cmp = p->trig_cmp;
    prm.trig_wait_value = p->trig_wait_value;
    prm.trig_wait_per_epoch = p->trig_wait_per_epoch;
    prm.trig_set_value = p->trig_set_value;
    prm.trig_set_per_epoch = p->trig_set_per_epoch;
    for (int r = 0; r < p->R; ++r) {
        prm.send[r] = sendbufs[r];
        prm.recv[r] = recvbufs[r];
    }
    return set_dispatch(p, prm);
}

static hccl_status_t check_buffers(hccl_plan_t* p, const void* const* sendbufs, void* const* recvbufs) {
    const int R = p->R;
    bool same = (int)p->checked_send.size() == R;
    for (int r = 0; same && r < R; ++r) same = p->checked_send[r] == sendbufs[r] && p->checked_recv[r] == recvbufs[r];
    if (same) return HCCL_OK;
    for (int r = 0; r < R; ++r) {
        if ((p->send_bytes[r] > 0 && !sendbufs[r]) || (p->recv_bytes[r] > 0 && !recvbufs[r])) return HCCL_ERR_INVALID_ARG;
        if (((uintptr_t)sendbufs[r] | (uintptr_t)recvbufs[r]) & (uintptr_t)(p->buf_align - 1)) return HCCL_ERR_ALIGNMENT;
    }
    // out-of-place only: no receive extent may intersect a send extent or another receive extent
    for (int d = 0; d < R; ++d) {
        const uintptr_t lo = (uintptr_t)recvbufs[d], hi = lo + (uintptr_t)p->recv_bytes[d];
        if (lo == hi) continue;
        for (int s = 0; s < R; ++s) {
            const uintptr_t slo = (uintptr_t)sendbufs[s], shi = slo + (uintptr_t)p->send_bytes[s];
            if (slo != shi && lo < shi && slo < hi) return HCCL_ERR_OVERLAP;
            if (s > d) {
                const uintptr_t rlo = (uintptr_t)recvbufs[s], rhi = rlo + (uintptr_t)p->recv_bytes[s];
                if (rlo != rhi && lo < rhi && rlo < hi) return HCCL_ERR_OVERLAP;
            }
        }
    }
    p->checked_send.assign(sendbufs, sendbufs + R);
    p->checked_recv.assign(recvbufs, recvbufs + R);
    return HCCL_OK;
}

hccl_status_t hccl_execute(hccl_plan_t* p, const void* const* sendbufs, void* const* recvbufs, void* stream) {
    if (!p || !sendbufs || !recvbufs) return HCCL_ERR_INVALID_ARG;
    if (!p->workspace) return HCCL_ERR_NOT_BOUND;
    hccl_status_t st = check_buffers(p, sendbufs, recvbufs);
    if (st != HCCL_OK) return st;
    if ((p->trig_wait_slot >= 0 || p->trig_set_slot >= 0) && !p->user_signals) return HCCL_ERR_INVALID_ARG;
    if (p->dynamic && p->dyn_device_tables) {
        // two launches: the table builder (one block per source rank), then the ordinary executor on what it wrote.
        // The builder holds the start gate; the executor behind it is ordered by the stream.
        if (!p->dyn_counts) return HCCL_ERR_INVALID_ARG;
        static thread_local PatchParams q;
        static thread_local ExecParams prm;
        char* ws = (char*)p->workspace;
        q.counts = (const long long*)p->dyn_counts;
        q.recvcounts_out = (long long*)p->dyn_recvcounts_out;
        q.rdispls_out = (long long*)p->dyn_rdispls_out;
        q.ctl = (Control*)(ws + p->layout.control);
        q.user_signals = (unsigned long long*)p->user_signals;
        q.descs = (Desc*)(ws + p->layout.descs);
        q.tiles = (Tile*)(ws + p->layout.tiles);
        q.R = (uint32_t)p->R;
        q.tile_cap = (uint32_t)p->tiles.size();
        q.end_tiles = p->dyn_end_tiles;
        q.timeout_ns = p->opts.timeout_ns;
        q.row_bytes = (unsigned long long)p->dyn_row_bytes;
        q.tile_bytes = p->opts.tile_bytes;
        q.trig_wait_slot = p->trig_wait_slot;
        q.trig_cmp = p->trig_cmp;
        q.trig_wait_value = p->trig_wait_value;
        q.trig_wait_per_epoch = p->trig_wait_per_epoch;
        for (int r = 0; r < p->R; ++r) {
            q.max_send_rows[r] = p->dyn_max_send_rows[r];
            q.max_recv_rows[r] = p->dyn_max_recv_rows[r];
        }
        hccl_a2a_patch<<<p->R, 256, 0, (cudaStream_t)stream>>>(q);
        CUDA_TRY(cudaGetLastError());
        const int blocks = fill_params(p, prm, sendbufs, recvbufs);
        prm.trig_wait_slot = -1;   // the builder has waited already
        prm.static_tickets = 0;    // how many items are real is known only on the device: tickets and END markers
        if (p->opts.engine == HCCL_ENGINE_BULK) {
            const bulk::StageConfig sc = bulk::stage_config(p->opts.stages, p->opts.stage_kib);
            hccl_executor_bulk<<<blocks, std::max(128, p->opts.threads), sc.smem, (cudaStream_t)stream>>>(
                prm, sc.ns, (uint32_t)(p->opts.copy_by_warps == 1 || (p->opts.copy_by_warps == 0 && p->opts.sm_budget < 100)), sc.stage_bytes);
        } else if (p->opts.light) {
            hccl_executor_lsu_light<<<blocks, p->opts.threads, 0, (cudaStream_t)stream>>>(prm);
        } else {
            hccl_executor_lsu<<<blocks, p->opts.threads, 0, (cudaStream_t)stream>>>(prm);
        }
        CUDA_TRY(cudaGetLastError());
        p->epoch += 1;
        return HCCL_OK;
    }
    if (p->dynamic) {
        if (!p->dyn_counts) return HCCL_ERR_INVALID_ARG;
        static thread_local DynParams q;
        const uint32_t epoch = p->epoch + 1;
        q.counts = (const long long*)p->dyn_counts;
        q.recvcounts_out = (long long*)p->dyn_recvcounts_out;
        q.rdispls_out = (long long*)p->dyn_rdispls_out;
        q.ctl = (Control*)((char*)p->workspace + p->layout.control);
        q.user_signals = (unsigned long long*)p->user_signals;
        q.R = (uint32_t)p->R;
        q.nblocks = (uint32_t)p->opts.sm_budget;
        q.timeout_ns = p->opts.timeout_ns;
        q.row_bytes = (unsigned long long)p->dyn_row_bytes;
        q.tile_bytes = p->opts.tile_bytes;
        q.trig_wait_slot = p->trig_wait_slot;
        q.trig_set_slot = p->trig_set_slot;
        q.trig_cmp = p->trig_cmp;
        q.trig_wait_value = p->trig_wait_value;
        q.trig_wait_per_epoch = p->trig_wait_per_epoch;
        q.trig_set_value = p->trig_set_value;
        q.trig_set_per_epoch = p->trig_set_per_epoch;
        for (int r = 0; r < p->R; ++r) {
            q.max_send_rows[r] = p->dyn_max_send_rows[r];
            q.max_recv_rows[r] = p->dyn_max_recv_rows[r];
            q.send[r] = sendbufs[r];
            q.recv[r] = recvbufs[r];
        }
        const size_t RR = (size_t)p->R * p->R;
        const size_t smem = RR * 24 + (RR + 1) * 4 + 16;
        hccl_a2a_dynamic<<<p->opts.sm_budget, p->opts.threads, smem, (cudaStream_t)stream>>>(q);
        CUDA_TRY(cudaGetLastError());
        p->epoch = epoch;
        return HCCL_OK;
    }
    static thread_local ExecParams prm;  // 4 KB+: keep it off the stack
    const uint32_t epoch = p->epoch + 1;
    const int blocks = fill_params(p, prm, sendbufs, recvbufs);
    if (p->opts.engine == HCCL_ENGINE_BULK && p->chain_len) {
        // stages sized for the widest operand that arrives through them (B of every step, A of a chain's first)
        const bool wide = p->chain_wide;
        if (p->chain_copies) hccl_executor_chain<<<blocks, CHAIN_THREADS, CHAIN_SMEM_BYTES, (cudaStream_t)stream>>>(prm, wide ? 3u : 6u, CHAIN_PIECE_ELEMS * (wide ? 4u : 2u));
        else hccl_executor_chain_sums<<<blocks, CHAIN_THREADS, CHAIN_SMEM_BYTES, (cudaStream_t)stream>>>(prm, wide ? 3u : 6u, CHAIN_PIECE_ELEMS * (wide ? 4u : 2u));
    } else if (p->opts.engine == HCCL_ENGINE_BULK) {
        const bulk::StageConfig sc = bulk::stage_config(p->opts.stages, p->opts.stage_kib);
        const int threads = std::max(128, p->opts.threads);
        hccl_executor_bulk<<<blocks, threads, sc.smem, (cudaStream_t)stream>>>(prm, sc.ns, (uint32_t)(p->opts.copy_by_warps == 1 || (p->opts.copy_by_warps == 0 && p->opts.sm_budget < 100)),
                                                                              sc.stage_bytes);
    } else {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3((unsigned)p->opts.threads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = (cudaStream_t)stream;
        cudaLaunchAttribute attr[1];
        int nattr = 0;
        if (p->opts.cluster > 1 && blocks % p->opts.cluster == 0) {
            // blocks of one cluster are placed on SMs of one GPC next to each other: a budget of B blocks then
            // takes B / cluster neighbourhoods away from a concurrent kernel instead of B scattered SMs
            attr[nattr].id = cudaLaunchAttributeClusterDimension;
            attr[nattr].val.clusterDim.x = (unsigned)p->opts.cluster;
            attr[nattr].val.clusterDim.y = 1;
            attr[nattr].val.clusterDim.z = 1;
            ++nattr;
        }
        cfg.attrs = attr;
        cfg.numAttrs = (unsigned)nattr;
        if (p->opts.light)
            CUDA_TRY(cudaLaunchKernelEx(&cfg, hccl_executor_lsu_light, prm));
        else
            CUDA_TRY(cudaLaunchKernelEx(&cfg, hccl_executor_lsu, prm));
    }
    CUDA_TRY(cudaGetLastError());
    p->epoch = epoch;
    return HCCL_OK;
}

hccl_status_t hccl_execute_host(hccl_plan_t* p, const void* const* host_send, void* const* host_recv, void* const* dev_send,
                                void* const* dev_recv, void* stream) {
    if (!p || !host_send || !host_recv || !dev_send || !dev_recv) return HCCL_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    for (int r = 0; r < p->R; ++r)
        if (p->send_bytes[r] > 0) CUDA_TRY(cudaMemcpyAsync(dev_send[r], host_send[r], (size_t)p->send_bytes[r], cudaMemcpyHostToDevice, s));
    hccl_status_t st = hccl_execute(p, (const void* const*)dev_send, dev_recv, stream);
    if (st != HCCL_OK) return st;
    for (int r = 0; r < p->R; ++r)
        if (p->recv_bytes[r] > 0) CUDA_TRY(cudaMemcpyAsync(host_recv[r], dev_recv[r], (size_t)p->recv_bytes[r], cudaMemcpyDeviceToHost, s));
    return HCCL_OK;
}

// ---------------------------------------------------------------------- host pipeline (AllToAllv by destination windows)
}  // extern "C"

struct hccl_hostpipe {
    int R = 0;
    int64_t row_bytes = 0;
    std::vector<int64_t> counts;          // [s*R+d] rows
    std::vector<int64_t> sdispl;          // packed, rows
    std::vector<int64_t> recv_rows;       // per destination
    std::vector<int32_t> first_dest;      // n_windows + 1
    std::vector<hccl_plan_t*> plans;      // one per window
    std::vector<size_t> ws_off;           // each sub-plan's slice of the workspace
    size_t ws_total = 0;
    std::vector<cudaEvent_t> in_done, exec_done, out_done;
    cudaEvent_t all_done = nullptr;
    bool bound = false, ran = false;
    ~hccl_hostpipe() {
        for (hccl_plan_t* q : plans) hccl_plan_destroy(q);
        for (cudaEvent_t e : in_done) cudaEventDestroy(e);
        for (cudaEvent_t e : exec_done) cudaEventDestroy(e);
        for (cudaEvent_t e : out_done) cudaEventDestroy(e);
        if (all_done) cudaEventDestroy(all_done);
    }
};

extern "C" {

hccl_status_t hccl_hostpipe_alltoallv_create(int R, const int64_t* sendcounts, hccl_dtype_t dt, int64_t row_elems, int n_windows,
                                             const hccl_opts_t* opts, hccl_hostpipe_t** out) {
    if (!out || !sendcounts || R < 1 || R > HCCL_MAX_RANKS || row_elems < 1 || n_windows < 1) return HCCL_ERR_INVALID_ARG;
    if (dt != HCCL_FP32 && dt != HCCL_BF16 && dt != HCCL_FP16) return HCCL_ERR_DTYPE;
    hccl_hostpipe* hp = new (std::nothrow) hccl_hostpipe();
    if (!hp) return HCCL_ERR_INVALID_ARG;
    hp->R = R;
    hp->row_bytes = row_elems * (dt == HCCL_FP32 ? 4 : 2);
    hp->counts.assign(sendcounts, sendcounts + (size_t)R * R);
    hp->sdispl.assign((size_t)R * R, 0);
    hp->recv_rows.assign(R, 0);
    int64_t total = 0;
    for (int s = 0; s < R; ++s) {
        int64_t acc = 0;
        for (int d = 0; d < R; ++d) {
            const int64_t c = sendcounts[(size_t)s * R + d];
            if (c < 0) {
                delete hp;
                return HCCL_ERR_INVALID_ARG;
            }
            hp->sdispl[(size_t)s * R + d] = acc;
            acc += c;
            hp->recv_rows[d] += c;
            total += c;
        }
    }
    // Contiguous windows of destinations, each closed once the rows received so far reach its cumulative
    // share. The shares taper towards both ends (weights 1, 2, 3, 4, 4, ..., 4, 3, 2, 1): the first copy-in
    // and the last copy-out are the only steps nothing overlaps, so those windows are the small ones.
    const int W = std::min(n_windows, R);
    std::vector<int64_t> cum(W + 1, 0);
    for (int g = 0; g < W; ++g) cum[g + 1] = cum[g] + std::min(std::min(g + 1, W - g), 4);
    hp->first_dest.push_back(0);
    int64_t acc = 0, in_window = 0;
    for (int d = 0; d < R; ++d) {
        acc += hp->recv_rows[d];
        in_window += hp->recv_rows[d];
        const int made = (int)hp->first_dest.size();  // windows closed so far + 1
        if (made < W && (__int128)acc * cum[W] >= (__int128)total * cum[made] && in_window > 0 && d + 1 < R) {
            hp->first_dest.push_back(d + 1);
            in_window = 0;
        }
    }
    hp->first_dest.push_back(R);
    // a trailing window without rows joins the one before it
    while (hp->first_dest.size() > 2) {
        int64_t rows = 0;
        for (int d = hp->first_dest[hp->first_dest.size() - 2]; d < R; ++d) rows += hp->recv_rows[d];
        if (rows > 0) break;
        hp->first_dest.erase(hp->first_dest.end() - 2);
    }
    const int nw = (int)hp->first_dest.size() - 1;
    for (int g = 0; g < nw; ++g) {
        hccl_plan_t* q = nullptr;
        hccl_status_t st = hccl::plan_alltoallv_window(R, sendcounts, nullptr, nullptr, nullptr, dt, row_elems, opts,
                                                       hp->first_dest[g], hp->first_dest[g + 1], &q);
        if (st != HCCL_OK) {
            delete hp;
            return st;
        }
        hp->plans.push_back(q);
        hp->ws_off.push_back(hp->ws_total);
        hp->ws_total += (size_t)((q->layout.total + 255) / 256 * 256);
    }
    *out = hp;
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_windows(const hccl_hostpipe_t* hp, int32_t* n_windows, int32_t* first_dest) {
    if (!hp || !n_windows) return HCCL_ERR_INVALID_ARG;
    *n_windows = (int32_t)hp->plans.size();
    if (first_dest)
        for (size_t i = 0; i < hp->first_dest.size(); ++i) first_dest[i] = hp->first_dest[i];
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_workspace_bytes(const hccl_hostpipe_t* hp, size_t* bytes) {
    if (!hp || !bytes) return HCCL_ERR_INVALID_ARG;
    *bytes = hp->ws_total;
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_bind(hccl_hostpipe_t* hp, void* dev_workspace, size_t bytes, void* stream) {
    if (!hp || !dev_workspace) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)dev_workspace) % 256) return HCCL_ERR_ALIGNMENT;
    if (bytes < hp->ws_total) return HCCL_ERR_WORKSPACE;
    for (size_t g = 0; g < hp->plans.size(); ++g) {
        hccl_status_t st = hccl_plan_bind(hp->plans[g], (char*)dev_workspace + hp->ws_off[g], (size_t)hp->plans[g]->layout.total, stream);
        if (st != HCCL_OK) return st;
    }
    if (!hp->all_done) {
        hp->in_done.resize(hp->plans.size());
        hp->exec_done.resize(hp->plans.size());
        hp->out_done.resize(hp->plans.size());
        for (size_t g = 0; g < hp->plans.size(); ++g) {
            CUDA_TRY(cudaEventCreateWithFlags(&hp->in_done[g], cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&hp->exec_done[g], cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&hp->out_done[g], cudaEventDisableTiming));
        }
        CUDA_TRY(cudaEventCreateWithFlags(&hp->all_done, cudaEventDisableTiming));
    }
    hp->bound = true;
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_execute(hccl_hostpipe_t* hp, const void* const* host_send, void* const* host_recv, void* const* dev_send,
                                    void* const* dev_recv, void* stream_in, void* stream_exec, void* stream_out) {
    if (!hp || !host_send || !host_recv || !dev_send || !dev_recv) return HCCL_ERR_INVALID_ARG;
    if (!hp->bound) return HCCL_ERR_NOT_BOUND;
    cudaStream_t si = (cudaStream_t)stream_in, sx = (cudaStream_t)stream_exec, so = (cudaStream_t)stream_out;
    const int R = hp->R;
    // The staging buffers are reused by the next call. Its copies-in may start once the previous call's last
    // exchange has run (nothing reads the send staging after that), and its exchange of window g once the
    // previous call's copy-out of window g has finished; so one call's drain overlaps the next one's fill.
    if (hp->ran) CUDA_TRY(cudaStreamWaitEvent(si, hp->exec_done.back(), 0));
    for (size_t g = 0; g < hp->plans.size(); ++g) {
        const int d0 = hp->first_dest[g], d1 = hp->first_dest[g + 1];
        for (int s = 0; s < R; ++s) {  // rows of source s bound for destinations d0..d1-1: one contiguous slice
            const int64_t lo = hp->sdispl[(size_t)s * R + d0];
            const int64_t hi = d1 < R ? hp->sdispl[(size_t)s * R + d1] : hp->sdispl[(size_t)s * R + R - 1] + hp->counts[(size_t)s * R + R - 1];
            if (hi > lo)
                CUDA_TRY(cudaMemcpyAsync((char*)dev_send[s] + lo * hp->row_bytes, (const char*)host_send[s] + lo * hp->row_bytes,
                                         (size_t)((hi - lo) * hp->row_bytes), cudaMemcpyHostToDevice, si));
        }
        CUDA_TRY(cudaEventRecord(hp->in_done[g], si));
        CUDA_TRY(cudaStreamWaitEvent(sx, hp->in_done[g], 0));
        if (hp->ran) CUDA_TRY(cudaStreamWaitEvent(sx, hp->out_done[g], 0));
        hccl_status_t st = hccl_execute(hp->plans[g], (const void* const*)dev_send, dev_recv, stream_exec);
        if (st != HCCL_OK) return st;
        CUDA_TRY(cudaEventRecord(hp->exec_done[g], sx));
        CUDA_TRY(cudaStreamWaitEvent(so, hp->exec_done[g], 0));
        for (int d = d0; d < d1; ++d)
            if (hp->recv_rows[d] > 0)
                CUDA_TRY(cudaMemcpyAsync(host_recv[d], dev_recv[d], (size_t)(hp->recv_rows[d] * hp->row_bytes), cudaMemcpyDeviceToHost, so));
        CUDA_TRY(cudaEventRecord(hp->out_done[g], so));
    }
    CUDA_TRY(cudaEventRecord(hp->all_done, so));
    hp->ran = true;
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_status(hccl_hostpipe_t* hp, hccl_status_t* device_status, int64_t* detail) {
    if (!hp || !device_status) return HCCL_ERR_INVALID_ARG;
    if (!hp->bound) return HCCL_ERR_NOT_BOUND;
    *device_status = HCCL_OK;
    for (hccl_plan_t* q : hp->plans) {
        hccl_status_t ds = HCCL_OK;
        int64_t dd = 0;
        hccl_status_t st = hccl_plan_status(q, &ds, &dd);
        if (st != HCCL_OK) return st;
        if (ds != HCCL_OK) {
            *device_status = ds;
            if (detail) *detail = dd;
            return HCCL_OK;
        }
    }
    if (detail) *detail = 0;
    return HCCL_OK;
}

void hccl_hostpipe_destroy(hccl_hostpipe_t* hp) { delete hp; }

hccl_status_t hccl_plan_status(hccl_plan_t* p, hccl_status_t* device_status, int64_t* detail) {
    if (!p || !device_status) return HCCL_ERR_INVALID_ARG;
    if (!p->workspace) return HCCL_ERR_NOT_BOUND;
    Control c;
    CUDA_TRY(cudaMemcpy(&c, (char*)p->workspace + p->layout.control, sizeof(c), cudaMemcpyDeviceToHost));
    // The device numbers its own executions (so that graph replays count too): the last one failed if the
    // failure stamp carries its number.
    if (c.done_epoch != 0 && c.fail_epoch == c.done_epoch) {
        *device_status = (hccl_status_t)c.status;
        if (detail) *detail = (int64_t)c.detail;
        return HCCL_OK;
    }
    if (c.exits != 0) return HCCL_ERR_BUSY;  // blocks of an execution are still leaving: synchronise first
    *device_status = HCCL_OK;
    if (detail) *detail = (int64_t)c.done_epoch;
    return HCCL_OK;
}

}  // extern "C"

// ====================================================================== resident executor: host side
extern "C" {

hccl_status_t hccl_server_start(hccl_plan_t* p, const void* const* sendbufs, void* const* recvbufs, void* host_doorbell,
                                uint64_t idle_timeout_ns, void* stream) {
    if (!p || !sendbufs || !recvbufs || !host_doorbell) return HCCL_ERR_INVALID_ARG;
    if (!p->workspace) return HCCL_ERR_NOT_BOUND;
    if (p->dynamic || p->server_db) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)host_doorbell) % 64) return HCCL_ERR_ALIGNMENT;
    hccl_status_t st = check_buffers(p, sendbufs, recvbufs);
    if (st != HCCL_OK) return st;
    void* dev_db = nullptr;
    CUDA_TRY(cudaHostGetDevicePointer(&dev_db, host_doorbell, 0));  // fails unless the record is pinned, mapped memory
    cudaStream_t s = (cudaStream_t)stream;
    Control c;
    CUDA_TRY(cudaStreamSynchronize(s));
    CUDA_TRY(cudaMemcpy(&c, (char*)p->workspace + p->layout.control, sizeof(c), cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemsetAsync((char*)p->workspace + p->layout.control + offsetof(Control, server_go), 0, 4, s));
    std::memset(host_doorbell, 0, sizeof(Doorbell));
    static thread_local ExecParams prm;
    if (p->opts.quantum > 0) return HCCL_ERR_INVALID_ARG;  // resident blocks are persistent by definition
    const int blocks = fill_params(p, prm, sendbufs, recvbufs);
    // every block must be resident at once (the blocks wait for each other between executions)
    int dev = 0, sms = 0, per_sm = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, hccl_executor_resident, p->opts.threads, 0));
    if (blocks > sms * per_sm) return HCCL_ERR_INVALID_ARG;
    Doorbell* db = (Doorbell*)dev_db;
    unsigned long long idle = idle_timeout_ns ? idle_timeout_ns : 100000000ull;
    uint32_t first_epoch = c.done_epoch + 1;
    prm.host_completed = &db->completed;
    prm.host_t_done = &db->t_done_ns;
    prm.first_epoch = first_epoch;
    void* args[] = {(void*)&prm, (void*)&db, (void*)&idle, (void*)&first_epoch};
    CUDA_TRY(cudaLaunchCooperativeKernel((const void*)hccl_executor_resident, dim3((unsigned)blocks), dim3((unsigned)p->opts.threads), args, 0, s));
    p->server_db = host_doorbell;
    p->server_rings = 0;
    return HCCL_OK;
}

hccl_status_t hccl_server_ring(hccl_plan_t* p) {
    if (!p || !p->server_db) return HCCL_ERR_INVALID_ARG;
    volatile Doorbell* db = (volatile Doorbell*)p->server_db;
    if (db->exited) return db->exited == 3 ? (hccl_status_t)db->status : HCCL_ERR_TIMEOUT;  // the kernel has left: start it again
    std::atomic_thread_fence(std::memory_order_release);
    db->request = ++p->server_rings;
    return HCCL_OK;
}

hccl_status_t hccl_server_wait(hccl_plan_t* p, uint64_t timeout_ns) {
    if (!p || !p->server_db) return HCCL_ERR_INVALID_ARG;
    volatile Doorbell* db = (volatile Doorbell*)p->server_db;
    const auto t0 = std::chrono::steady_clock::now();
    const uint64_t limit = timeout_ns ? timeout_ns : 5000000000ull;
    for (;;) {
        if (db->completed >= p->server_rings) break;
        if (db->exited) break;
        if ((uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count() > limit) return HCCL_ERR_TIMEOUT;
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    if (db->exited == 3) return (hccl_status_t)db->status;
    if (db->completed < p->server_rings) return HCCL_ERR_TIMEOUT;  // left (idle or stopped) before serving this ring
    return HCCL_OK;
}

hccl_status_t hccl_server_stop(hccl_plan_t* p) {
    if (!p || !p->server_db) return HCCL_ERR_INVALID_ARG;
    volatile Doorbell* db = (volatile Doorbell*)p->server_db;
    db->stop = 1;
    p->epoch += p->server_rings;
    p->server_db = nullptr;
    return HCCL_OK;
}

}  // extern "C"

// ====================================================================== execution without any allocation
// Workspace for callers that cannot obtain device memory of their own: one array that lives in the
// library's device image for the life of the process (every GPU that loads the library holds it).
#define HCCL_NOALLOC_WORKSPACE_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_noalloc_workspace[HCCL_NOALLOC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_noalloc_addr[kMaxDevices] = {};  // device address of g_noalloc_workspace, per device ordinal
std::mutex g_noalloc_mu;
}  // namespace

extern "C" hccl_status_t hccl_execute_noalloc(hccl_plan_t* p, const void* const* sendbufs, void* const* recvbufs, void* stream) {
    if (!p || !sendbufs || !recvbufs) return HCCL_ERR_INVALID_ARG;
    if (p->layout.total > HCCL_NOALLOC_WORKSPACE_BYTES) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "plan needs %llu workspace bytes; the built-in workspace holds %u",
                 (unsigned long long)p->layout.total, HCCL_NOALLOC_WORKSPACE_BYTES);
        return HCCL_ERR_WORKSPACE;
    }
    if (p->trig_wait_slot >= 0 || p->trig_set_slot >= 0 || p->dynamic) return HCCL_ERR_INVALID_ARG;  // triggers and device-resident plans belong to bound plans
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return HCCL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_noalloc_mu);  // one user of the array at a time from this process
    if (!g_noalloc_addr[dev]) {
        // In host code the array's name is only a handle; its device address on the current device is
        // looked up once here and that address is what the kernel receives.
        void* ptr = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_workspace));
        if (!ptr || ((uintptr_t)ptr % 256) != 0) return HCCL_ERR_ALIGNMENT;
        g_noalloc_addr[dev] = ptr;
    }
    char* ws = (char*)g_noalloc_addr[dev];
    // same aliasing rules as hccl_execute, checked on every call (nothing is cached for this path)
    const int R = p->R;
    for (int r = 0; r < R; ++r) {
        if ((p->send_bytes[r] > 0 && !sendbufs[r]) || (p->recv_bytes[r] > 0 && !recvbufs[r])) return HCCL_ERR_INVALID_ARG;
        if (((uintptr_t)sendbufs[r] | (uintptr_t)recvbufs[r]) & (uintptr_t)(p->buf_align - 1)) return HCCL_ERR_ALIGNMENT;
    }
    for (int d = 0; d < R; ++d) {
        const uintptr_t lo = (uintptr_t)recvbufs[d], hi = lo + (uintptr_t)p->recv_bytes[d];
        if (lo == hi) continue;
        for (int s = 0; s < R; ++s) {
            const uintptr_t slo = (uintptr_t)sendbufs[s], shi = slo + (uintptr_t)p->send_bytes[s];
            if (slo != shi && lo < shi && slo < hi) return HCCL_ERR_OVERLAP;
            const uintptr_t rlo = (uintptr_t)recvbufs[s], rhi = rlo + (uintptr_t)p->recv_bytes[s];
            if (s > d && rlo != rhi && lo < rhi && rlo < hi) return HCCL_ERR_OVERLAP;
        }
    }
    // The array keeps whatever the previous call left. Everything that must start at zero (control words,
    // dependency counters, signal slots) is rewritten together with this plan's tables; the FP32 scratch
    // behind them is always written before it is read within one execution, so it is left as it is.
    const Layout& L = p->layout;
    static thread_local std::vector<char> img;
    img.assign((size_t)L.scratch, 0);
    if (!p->descs.empty()) std::memcpy(img.data() + L.descs, p->descs.data(), p->descs.size() * sizeof(Desc));
    if (!p->tiles.empty()) std::memcpy(img.data() + L.tiles, p->tiles.data(), p->tiles.size() * sizeof(Tile));
    if (!p->waits.empty()) std::memcpy(img.data() + L.waits, p->waits.data(), p->waits.size() * sizeof(Wait));
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(cudaMemcpyAsync(ws, img.data(), img.size(), cudaMemcpyHostToDevice, st));
    static thread_local ExecParams prm;
    prm.descs = (const Desc*)(ws + L.descs);
    prm.tiles = (const Tile*)(ws + L.tiles);
    prm.waits = (const Wait*)(ws + L.waits);
    prm.counters = (uint32_t*)(ws + L.counters);
    prm.signals = (unsigned long long*)(ws + L.signals);
    prm.ctl = (Control*)(ws + L.control);
    prm.scratch = ws + L.scratch;
    prm.user_signals = nullptr;
    prm.trace = nullptr;
    prm.trace_cap = 0;
    prm.n_tiles = (uint32_t)p->tiles.size();
    prm.n_descs = (uint32_t)p->descs.size();
    prm.n_syncs = (uint32_t)p->sync_per_epoch.size();
    prm.n_waits = (uint32_t)p->waits.size();
    prm.n_signals = (uint32_t)p->n_signals;
    prm.R = (uint32_t)R;
    prm.timeout_ns = p->opts.timeout_ns;
    prm.n_user_signals = 0;
    prm.trig_wait_slot = -1;
    prm.trig_set_slot = -1;
    prm.trig_cmp = 0;
    prm.trig_wait_value = prm.trig_set_value = prm.trig_wait_per_epoch = prm.trig_set_per_epoch = 0;
    for (int r = 0; r < R; ++r) {
        prm.send[r] = sendbufs[r];
        prm.recv[r] = recvbufs[r];
    }
    const int blocks = set_dispatch(p, prm);
    hccl_executor_lsu<<<blocks, p->opts.threads, 0, st>>>(prm);
    CUDA_TRY(cudaGetLastError());
    // This call owns the shared array until its kernel is done, so it waits here and hands back the
    // device-side verdict itself.
    CUDA_TRY(cudaStreamSynchronize(st));
    Control c;
    CUDA_TRY(cudaMemcpy(&c, ws + L.control, sizeof(c), cudaMemcpyDeviceToHost));
    if (c.fail_epoch == 1) return (hccl_status_t)c.status;
    if (c.done_epoch != 1) return HCCL_ERR_BUSY;
    return HCCL_OK;
}
