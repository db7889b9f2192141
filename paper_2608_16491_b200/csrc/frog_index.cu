// Index handle: file parsing, device residency (paper Sec. 8.1.3: index and vectors stay in GPU
// memory), error strings, and the host-buffer search call that includes the transfers.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "frog_internal.h"

namespace {

thread_local int g_last_cuda_error = 0;

struct FileHeader {
    uint32_t version, d, d_pad, H, m, n_inv, ef_c, patience;
    float beta, gamma;
    uint64_t n, seed;
    uint32_t bot, reserved;
    uint64_t off_attr, off_r2i, off_vec, off_enc, file_bytes;
};

int parse_header(const unsigned char* h, FileHeader* out) {
    if (std::memcmp(h, "FROGIDX1", 8) != 0) return FROG_ERR_FORMAT;
    std::memcpy(&out->version, h + 8, 32);
    std::memcpy(&out->beta, h + 40, 8);
    std::memcpy(&out->n, h + 48, 16);
    std::memcpy(&out->bot, h + 64, 8);
    std::memcpy(&out->off_attr, h + 72, 40);
    if (out->version != 1 || out->bot != 0xFFFFFFFFu) return FROG_ERR_FORMAT;
    if (out->n < 1 || out->n >= 0x7FFFFFFFull) return FROG_ERR_FORMAT;
    if (out->d < 1 || out->d_pad != (out->d + 3) / 4 * 4) return FROG_ERR_FORMAT;
    if (out->H < 1 || out->H > 40 || out->m < 1 || out->m > 1024) return FROG_ERR_FORMAT;
    const uint64_t n = out->n;
    if ((out->off_attr | out->off_r2i | out->off_vec | out->off_enc) & 127ull) return FROG_ERR_FORMAT;
    if (out->off_attr < 256 || out->off_r2i < out->off_attr + n * 4 || out->off_vec < out->off_r2i + n * 4 ||
        out->off_enc < out->off_vec + n * out->d_pad * 4 ||
        out->file_bytes != out->off_enc + n * out->H * out->m * 4)
        return FROG_ERR_FORMAT;
    return FROG_OK;
}

int alloc_device(frog_index* ix) {
    const frog_index_info_t& I = ix->info;
    const size_t n = (size_t)I.n;
    const size_t b_attr = n * 4, b_vec = n * (size_t)I.d_pad * 4, b_enc = n * (size_t)I.H * I.m * 4;
    cudaError_t e;
    if ((e = cudaMalloc(&ix->d_sorted_attr, b_attr)) != cudaSuccess ||
        (e = cudaMalloc(&ix->d_rank2id, b_attr)) != cudaSuccess ||
        (e = cudaMalloc(&ix->d_vectors, b_vec)) != cudaSuccess ||
        (e = cudaMalloc(&ix->d_enc, b_enc)) != cudaSuccess) {
        froghost::set_cuda_error(e);
        return e == cudaErrorMemoryAllocation ? FROG_ERR_NOMEM : FROG_ERR_CUDA;
    }
    ix->info.device_bytes = (int64_t)(2 * b_attr + b_vec + b_enc);
    cudaDeviceProp prop;
    FROG_CUDA_TRY(cudaGetDeviceProperties(&prop, I.device));
    ix->sm_count = prop.multiProcessorCount;
    ix->has_tmap_f32 = froghost::make_row_tensor_map(ix->d_vectors, false, I.d_pad, (size_t)I.d_pad * 4, n, &ix->tmap_f32);
    return FROG_OK;
}

// read `bytes` at file offset `off` and copy them to device memory through a pinned bounce buffer
int stream_to_device(FILE* f, uint64_t off, size_t bytes, void* dst) {
    const size_t CH = (size_t)64 << 20;
    void* bounce = nullptr;
    FROG_CUDA_TRY(cudaMallocHost(&bounce, CH));
    int rc = FROG_OK;
    if (fseeko(f, (off_t)off, SEEK_SET) != 0) rc = FROG_ERR_IO;
    size_t done = 0;
    while (rc == FROG_OK && done < bytes) {
        size_t c = bytes - done < CH ? bytes - done : CH;
        if (fread(bounce, 1, c, f) != c) { rc = FROG_ERR_IO; break; }
        cudaError_t e = cudaMemcpy((char*)dst + done, bounce, c, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { froghost::set_cuda_error(e); rc = FROG_ERR_CUDA; break; }
        done += c;
    }
    cudaFreeHost(bounce);
    return rc;
}

}  // namespace

namespace froghost {
void set_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }
}  // namespace froghost

extern "C" int frog_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" const char* frog_strerror(int code) {
    switch (code) {
        case FROG_OK: return "ok";
        case FROG_ERR_INVALID_ARG: return "invalid argument";
        case FROG_ERR_IO: return "i/o error";
        case FROG_ERR_FORMAT: return "bad index file";
        case FROG_ERR_NOMEM: return "out of memory";
        case FROG_ERR_CUDA: return "CUDA error";
        case FROG_ERR_UNSUPPORTED: return "unsupported parameters";
        case FROG_ERR_TOO_LARGE: return "index too large for the static scratch (more than 2097152 objects)";
        default: return "unknown error";
    }
}

extern "C" void frog_index_free(frog_index_t* ix) {
    if (!ix) return;
    int dev_count = 0;
    if (cudaGetDeviceCount(&dev_count) == cudaSuccess && ix->info.device < dev_count) {
        cudaSetDevice(ix->info.device);
        cudaDeviceSynchronize();
        cudaFree(ix->d_sorted_attr);
        cudaFree(ix->d_rank2id);
        cudaFree(ix->d_vectors);
        cudaFree(ix->d_vectors_h);
        cudaFree(ix->d_enc);
        for (int i = 0; i < ix->n_scratch; ++i) {
            cudaFree(ix->scratch[i].d_work);
            cudaFree(ix->scratch[i].d_bitmap);
            cudaFree(ix->scratch[i].d_table);
            cudaFree(ix->scratch[i].d_plan);
            if (ix->scratch[i].done) cudaEventDestroy(ix->scratch[i].done);
            if (ix->scratch[i].k_begin) cudaEventDestroy(ix->scratch[i].k_begin);
            if (ix->scratch[i].k_end) cudaEventDestroy(ix->scratch[i].k_end);
        }
        cudaFree(ix->d_stage);
    }
    delete ix;
}

extern "C" int frog_index_info(const frog_index_t* ix, frog_index_info_t* out) {
    if (!ix || !out) return FROG_ERR_INVALID_ARG;
    *out = ix->info;
    return FROG_OK;
}

extern "C" int frog_index_load(const char* path, int device, frog_index_t** out) {
    if (!path || !out || device < 0) return FROG_ERR_INVALID_ARG;
    *out = nullptr;
    FILE* f = fopen(path, "rb");
    if (!f) return FROG_ERR_IO;
    unsigned char hdr[256];
    FileHeader fh;
    if (fread(hdr, 1, 256, f) != 256) { fclose(f); return FROG_ERR_FORMAT; }
    int rc = parse_header(hdr, &fh);
    if (rc == FROG_OK) {
        if (fseeko(f, 0, SEEK_END) != 0 || (uint64_t)ftello(f) != fh.file_bytes) rc = FROG_ERR_FORMAT;
    }
    if (rc != FROG_OK) { fclose(f); return rc; }
    int dev_count = 0;
    cudaError_t e = cudaGetDeviceCount(&dev_count);
    if (e != cudaSuccess) { froghost::set_cuda_error(e); fclose(f); return FROG_ERR_CUDA; }
    if (device >= dev_count) { fclose(f); return FROG_ERR_INVALID_ARG; }
    e = cudaSetDevice(device);
    if (e != cudaSuccess) { froghost::set_cuda_error(e); fclose(f); return FROG_ERR_CUDA; }

    frog_index* ix = new (std::nothrow) frog_index();
    if (!ix) { fclose(f); return FROG_ERR_NOMEM; }
    std::memset(&ix->info, 0, sizeof(ix->info));
    ix->info.n = (int64_t)fh.n;
    ix->info.d = (int32_t)fh.d;
    ix->info.d_pad = (int32_t)fh.d_pad;
    ix->info.H = (int32_t)fh.H;
    ix->info.m = (int32_t)fh.m;
    ix->info.n_inv = (int32_t)fh.n_inv;
    ix->info.ef_c = (int32_t)fh.ef_c;
    ix->info.patience = (int32_t)fh.patience;
    ix->info.beta = fh.beta;
    ix->info.gamma = fh.gamma;
    ix->info.seed = fh.seed;
    ix->info.device = device;
    rc = alloc_device(ix);
    const size_t n = (size_t)fh.n;
    if (rc == FROG_OK) rc = stream_to_device(f, fh.off_attr, n * 4, ix->d_sorted_attr);
    if (rc == FROG_OK) rc = stream_to_device(f, fh.off_r2i, n * 4, ix->d_rank2id);
    if (rc == FROG_OK) rc = stream_to_device(f, fh.off_vec, n * fh.d_pad * 4, ix->d_vectors);
    if (rc == FROG_OK) rc = stream_to_device(f, fh.off_enc, n * fh.H * fh.m * 4, ix->d_enc);
    fclose(f);
    if (rc != FROG_OK) { frog_index_free(ix); return rc; }
    *out = ix;
    return FROG_OK;
}

extern "C" int frog_index_from_host(const int32_t* sorted_attr, const int32_t* rank2id, const float* vectors,
                                    const uint32_t* enc, const frog_index_info_t* shape, int device,
                                    frog_index_t** out) {
    if (!sorted_attr || !rank2id || !vectors || !enc || !shape || !out || device < 0) return FROG_ERR_INVALID_ARG;
    *out = nullptr;
    if (shape->n < 1 || shape->n >= 0x7FFFFFFFll || shape->d < 1 || shape->d_pad != (shape->d + 3) / 4 * 4 ||
        shape->H < 1 || shape->H > 40 || shape->m < 1 || shape->m > 1024)
        return FROG_ERR_INVALID_ARG;
    int dev_count = 0;
    FROG_CUDA_TRY(cudaGetDeviceCount(&dev_count));
    if (device >= dev_count) return FROG_ERR_INVALID_ARG;
    FROG_CUDA_TRY(cudaSetDevice(device));
    frog_index* ix = new (std::nothrow) frog_index();
    if (!ix) return FROG_ERR_NOMEM;
    ix->info = *shape;
    ix->info.device = device;
    int rc = alloc_device(ix);
    const size_t n = (size_t)shape->n;
    cudaError_t e = cudaSuccess;
    if (rc == FROG_OK) {
        if ((e = cudaMemcpy(ix->d_sorted_attr, sorted_attr, n * 4, cudaMemcpyHostToDevice)) != cudaSuccess ||
            (e = cudaMemcpy(ix->d_rank2id, rank2id, n * 4, cudaMemcpyHostToDevice)) != cudaSuccess ||
            (e = cudaMemcpy(ix->d_vectors, vectors, n * (size_t)shape->d_pad * 4, cudaMemcpyHostToDevice)) != cudaSuccess ||
            (e = cudaMemcpy(ix->d_enc, enc, n * (size_t)shape->H * shape->m * 4, cudaMemcpyHostToDevice)) != cudaSuccess) {
            froghost::set_cuda_error(e);
            rc = FROG_ERR_CUDA;
        }
    }
    if (rc != FROG_OK) { frog_index_free(ix); return rc; }
    *out = ix;
    return FROG_OK;
}

extern "C" int frog_search_host(frog_index_t* ix, const float* queries, const int32_t* lo, const int32_t* hi,
                                int nq, int k, int beam_width, const frog_params_t* params,
                                int32_t* out_ids, float* out_dists, void* stream) {
    if (!ix || nq < 0) return FROG_ERR_INVALID_ARG;
    if (k < 1 || beam_width < 1 || beam_width > FROG_MAX_BEAM_WIDTH || k > beam_width) return FROG_ERR_INVALID_ARG;
    if (nq == 0) return FROG_OK;
    if (!queries || !lo || !hi || !out_ids || !out_dists) return FROG_ERR_INVALID_ARG;
    FROG_CUDA_TRY(cudaSetDevice(ix->info.device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Pinned (page-locked, device-mapped) host buffers need no staging: the kernels read each query
    // and write each result row across the bus themselves, so the transfers overlap the search
    // instead of bracketing it.  Pageable buffers take the staged path below.
    {
        const void* host[5] = {queries, lo, hi, out_ids, out_dists};
        void* dev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
        bool mapped = true;
        for (int i = 0; i < 5 && mapped; ++i) {
            cudaPointerAttributes at;
            if (cudaPointerGetAttributes(&at, host[i]) != cudaSuccess) { cudaGetLastError(); mapped = false; break; }
            mapped = at.type == cudaMemoryTypeHost && at.devicePointer != nullptr;
            dev[i] = at.devicePointer;
        }
        if (mapped) {
            int rc = frog_search_ex(ix, static_cast<const float*>(dev[0]), static_cast<const int32_t*>(dev[1]),
                                    static_cast<const int32_t*>(dev[2]), nq, k, beam_width, params,
                                    static_cast<int32_t*>(dev[3]), static_cast<float*>(dev[4]), nullptr, nullptr,
                                    nullptr, 0, stream);
            if (rc != FROG_OK) return rc;
            FROG_CUDA_TRY(cudaStreamSynchronize(s));
            return FROG_OK;
        }
    }
    std::lock_guard<std::mutex> stage_lock(ix->stage_mu);
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t b_q = up((size_t)nq * ix->info.d * 4), b_r = up((size_t)nq * 4), b_o = up((size_t)nq * k * 4);
    const size_t need = b_q + 2 * b_r + 2 * b_o;
    if (need > ix->stage_bytes) {
        FROG_CUDA_TRY(cudaStreamSynchronize(s));
        if (ix->d_stage) FROG_CUDA_TRY(cudaFree(ix->d_stage));
        ix->d_stage = nullptr;
        ix->stage_bytes = 0;
        cudaError_t e = cudaMalloc(&ix->d_stage, need);
        if (e != cudaSuccess) { froghost::set_cuda_error(e); return FROG_ERR_NOMEM; }
        ix->stage_bytes = need;
    }
    char* p = static_cast<char*>(ix->d_stage);
    float* d_q = reinterpret_cast<float*>(p);
    int32_t* d_lo = reinterpret_cast<int32_t*>(p + b_q);
    int32_t* d_hi = reinterpret_cast<int32_t*>(p + b_q + b_r);
    int32_t* d_ids = reinterpret_cast<int32_t*>(p + b_q + 2 * b_r);
    float* d_dist = reinterpret_cast<float*>(p + b_q + 2 * b_r + b_o);
    FROG_CUDA_TRY(cudaMemcpyAsync(d_q, queries, (size_t)nq * ix->info.d * 4, cudaMemcpyHostToDevice, s));
    FROG_CUDA_TRY(cudaMemcpyAsync(d_lo, lo, (size_t)nq * 4, cudaMemcpyHostToDevice, s));
    FROG_CUDA_TRY(cudaMemcpyAsync(d_hi, hi, (size_t)nq * 4, cudaMemcpyHostToDevice, s));
    int rc = frog_search_ex(ix, d_q, d_lo, d_hi, nq, k, beam_width, params, d_ids, d_dist, nullptr, nullptr,
                            nullptr, 0, stream);
    if (rc != FROG_OK) return rc;
    FROG_CUDA_TRY(cudaMemcpyAsync(out_ids, d_ids, (size_t)nq * k * 4, cudaMemcpyDeviceToHost, s));
    FROG_CUDA_TRY(cudaMemcpyAsync(out_dists, d_dist, (size_t)nq * k * 4, cudaMemcpyDeviceToHost, s));
    FROG_CUDA_TRY(cudaStreamSynchronize(s));
    return FROG_OK;
}
