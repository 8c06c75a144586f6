// Exchange memory of the real communication window: one block per rank (process, GPU) that holds
// the rank's two partial-sum buffers (window A: MLP partial sums; window B: attention partial sums),
// its arrival flags and its epoch counters.  Ranks learn each other's blocks either through CUDA IPC
// handles (one process per GPU; the handles travel over whatever channel the caller has - the
// Python layer uses torch.distributed) or, inside one process, as plain device pointers.
// The reduction itself is the window kernel's (window.cu): every rank reads every rank's buffer
// (Section 2, "Multi-device inference": one all-reduce per attention block and per MLP block).
#include <cuda_runtime.h>

#include <cstring>
#include <new>

#include "../../include/preserve.h"
#include "kernels.h"

using namespace prsv;

struct preserve_comm {
    int rank, n_ranks, max_batch, hidden, dev;
    uint8_t *block;                      // own block (cudaMalloc)
    size_t block_bytes, buf_bytes;
    uint8_t *peer[kMaxParts];            // every rank's block as seen from this process (own included)
    bool ipc_opened[kMaxParts];
};

namespace prsv {
constexpr size_t kCommHeaderBytes = 256;     // flags [2][kMaxParts] u32 (128 B), epoch[2], done[2]
uint32_t *comm_flags(uint8_t *block) { return reinterpret_cast<uint32_t *>(block); }
uint32_t *comm_epoch(uint8_t *block, int w) { return reinterpret_cast<uint32_t *>(block) + 2 * kMaxParts + w; }
unsigned *comm_done(uint8_t *block, int w) { return reinterpret_cast<unsigned *>(block) + 2 * kMaxParts + 2 + w; }

bool comm_fill(const preserve_comm *c, int window, CommView *v)
{
    if (!c)
        return false;
    for (int r = 0; r < c->n_ranks; ++r)
        if (!c->peer[r])
            return false;               // a peer has not been connected yet
    v->rank = c->rank;
    v->n_ranks = c->n_ranks;
    for (int r = 0; r < kMaxParts; ++r) {
        v->buf[r] = r < c->n_ranks ? c->peer[r] + kCommHeaderBytes + (size_t)window * c->buf_bytes : nullptr;
        v->flags[r] = r < c->n_ranks ? comm_flags(c->peer[r]) : nullptr;
    }
    v->epoch = comm_epoch(c->block, window);
    v->done = comm_done(c->block, window);
    return true;
}
int comm_hidden(const preserve_comm *c) { return c->hidden; }
int comm_max_batch(const preserve_comm *c) { return c->max_batch; }
}  // namespace prsv

extern "C" {

int preserve_comm_create(int32_t rank, int32_t n_ranks, int32_t max_batch, int32_t hidden, preserve_comm_t **out)
{
    if (out)
        *out = nullptr;
    if (!out || n_ranks < 1 || n_ranks > 8 || rank < 0 || rank >= n_ranks || max_batch < 1 || max_batch > 128 ||
        hidden < 128 || hidden % 128 || hidden > 16384)
        return PRESERVE_EINVAL;
    preserve_comm *c = new (std::nothrow) preserve_comm();
    if (!c)
        return PRESERVE_ENOMEM;
    c->rank = rank; c->n_ranks = n_ranks; c->max_batch = max_batch; c->hidden = hidden;
    if (cudaGetDevice(&c->dev) != cudaSuccess) {
        (void)cudaGetLastError();
        delete c;
        return PRESERVE_EARCH;
    }
    c->buf_bytes = ((size_t)max_batch * hidden * 2 + 255) & ~size_t(255);
    c->block_bytes = kCommHeaderBytes + 2 * c->buf_bytes;
    cudaError_t e = cudaMalloc(&c->block, c->block_bytes);
    if (e == cudaSuccess)
        e = cudaMemset(c->block, 0, c->block_bytes);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        if (c->block)
            cudaFree(c->block);
        delete c;
        return e == cudaErrorMemoryAllocation ? PRESERVE_ENOMEM : PRESERVE_ECUDA;
    }
    c->peer[rank] = c->block;
    *out = c;
    return PRESERVE_OK;
}

int preserve_comm_export(const preserve_comm_t *c, void *handle64)
{
    if (!c || !handle64)
        return PRESERVE_EINVAL;
    static_assert(sizeof(cudaIpcMemHandle_t) == 64, "IPC handle size");
    cudaIpcMemHandle_t h;
    if (cudaIpcGetMemHandle(&h, c->block) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    memcpy(handle64, &h, 64);
    return PRESERVE_OK;
}

int preserve_comm_import(preserve_comm_t *c, int32_t peer_rank, const void *handle64)
{
    if (!c || !handle64 || peer_rank < 0 || peer_rank >= c->n_ranks || peer_rank == c->rank || c->peer[peer_rank])
        return PRESERVE_EINVAL;
    cudaIpcMemHandle_t h;
    memcpy(&h, handle64, 64);
    void *p = nullptr;
    if (cudaSetDevice(c->dev) != cudaSuccess ||
        cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess || !p) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    c->peer[peer_rank] = static_cast<uint8_t *>(p);
    c->ipc_opened[peer_rank] = true;
    return PRESERVE_OK;
}

int preserve_comm_set_peer(preserve_comm_t *c, int32_t peer_rank, const preserve_comm_t *peer)
{
    if (!c || !peer || peer_rank < 0 || peer_rank >= c->n_ranks || peer_rank == c->rank || c->peer[peer_rank] ||
        peer->rank != peer_rank || peer->n_ranks != c->n_ranks || peer->block_bytes != c->block_bytes)
        return PRESERVE_EINVAL;
    c->peer[peer_rank] = peer->block;
    return PRESERVE_OK;
}

int preserve_comm_write(preserve_comm_t *c, int32_t window, const void *src_device, size_t bytes, void *cuda_stream)
{
    if (!c || !src_device || (window != 0 && window != 1) || bytes > c->buf_bytes)
        return PRESERVE_EINVAL;
    if (cudaMemcpyAsync(c->block + kCommHeaderBytes + (size_t)window * c->buf_bytes, src_device, bytes,
                        cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    return PRESERVE_OK;
}

int preserve_comm_debug_arrive(preserve_comm_t *c, int32_t window, int32_t from_rank, uint32_t epoch)
{
    if (!c || (window != 0 && window != 1) || from_rank < 0 || from_rank >= c->n_ranks)
        return PRESERVE_EINVAL;
    if (cudaSetDevice(c->dev) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(comm_flags(c->block) + window * kMaxParts + from_rank, &epoch, sizeof(epoch),
                   cudaMemcpyHostToDevice) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    return PRESERVE_OK;
}

int64_t preserve_comm_epoch(preserve_comm_t *c, int32_t window)
{
    if (!c || (window != 0 && window != 1))
        return -1;
    uint32_t e = 0;
    if (cudaSetDevice(c->dev) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(&e, comm_epoch(c->block, window), sizeof(e), cudaMemcpyDeviceToHost) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    return (int64_t)e;
}

void preserve_comm_destroy(preserve_comm_t *c)
{
    if (!c)
        return;
    cudaSetDevice(c->dev);
    cudaDeviceSynchronize();
    for (int r = 0; r < c->n_ranks; ++r)
        if (c->ipc_opened[r] && c->peer[r])
            cudaIpcCloseMemHandle(c->peer[r]);
    if (c->block)
        cudaFree(c->block);
    delete c;
}

}  // extern "C"
