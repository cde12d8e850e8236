// Page backends, physical page pool and per-tensor expert memory manager (Section 4.2).
#include "ew_vmm.h"

#include <cuda.h>
#include <cuda_runtime_api.h>

#include <algorithm>
#include <cstdio>

namespace ew {

// ------------------------------------------------------------------------------------------------
// CUDA driver backend.  Mapping of the paper's Table 2 onto the CUDA virtual memory API:
//   reserve address range -> cuMemAddressReserve      create / free a physical page -> cuMemCreate / cuMemRelease
//   map / unmap           -> cuMemMap (+ cuMemSetAccess) / cuMemUnmap
// ------------------------------------------------------------------------------------------------
namespace {

template <class F>
bool load_entry(const char *name, F *fn, std::string *err) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
        if (err) *err = std::string("driver entry point not found: ") + name;
        return false;
    }
    *fn = reinterpret_cast<F>(p);
    return true;
}

struct CudaBackend : PageBackend {
    int device = 0;
    CUresult (*pGranularity)(size_t *, const CUmemAllocationProp *, CUmemAllocationGranularity_flags) = nullptr;
    CUresult (*pReserve)(CUdeviceptr *, size_t, size_t, CUdeviceptr, unsigned long long) = nullptr;
    CUresult (*pAddrFree)(CUdeviceptr, size_t) = nullptr;
    CUresult (*pCreate)(CUmemGenericAllocationHandle *, size_t, const CUmemAllocationProp *, unsigned long long) = nullptr;
    CUresult (*pRelease)(CUmemGenericAllocationHandle) = nullptr;
    CUresult (*pMap)(CUdeviceptr, size_t, size_t, CUmemGenericAllocationHandle, unsigned long long) = nullptr;
    CUresult (*pSetAccess)(CUdeviceptr, size_t, const CUmemAccessDesc *, size_t) = nullptr;
    CUresult (*pUnmap)(CUdeviceptr, size_t) = nullptr;
    CUresult (*pErrStr)(CUresult, const char **) = nullptr;

    CUmemAllocationProp prop() const {
        CUmemAllocationProp p = {};
        p.type = CU_MEM_ALLOCATION_TYPE_PINNED;
        p.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
        p.location.id = device;
        return p;
    }
    int fail(const char *what, CUresult r) {
        const char *s = nullptr;
        if (pErrStr) pErrStr(r, &s);
        last_error = std::string(what) + ": " + (s ? s : "unknown driver error");
        return r == CUDA_ERROR_OUT_OF_MEMORY ? 2 : 6;
    }
    bool is_mock() const override { return false; }
    int granularity(size_t *g) override {
        CUmemAllocationProp p = prop();
        CUresult r = pGranularity(g, &p, CU_MEM_ALLOC_GRANULARITY_MINIMUM);
        return r == CUDA_SUCCESS ? 0 : fail("cuMemGetAllocationGranularity", r);
    }
    int reserve(size_t bytes, size_t align, uint64_t *va) override {
        CUdeviceptr p = 0;
        CUresult r = pReserve(&p, bytes, align, 0, 0);
        if (r != CUDA_SUCCESS) return fail("cuMemAddressReserve", r);
        *va = (uint64_t)p;
        return 0;
    }
    int free_va(uint64_t va, size_t bytes) override {
        CUresult r = pAddrFree((CUdeviceptr)va, bytes);
        return r == CUDA_SUCCESS ? 0 : fail("cuMemAddressFree", r);
    }
    int create(size_t bytes, uint64_t *handle) override {
        CUmemAllocationProp p = prop();
        CUmemGenericAllocationHandle h = 0;
        CUresult r = pCreate(&h, bytes, &p, 0);
        if (r != CUDA_SUCCESS) return fail("cuMemCreate", r);
        *handle = (uint64_t)h;
        return 0;
    }
    int release(uint64_t handle) override {
        CUresult r = pRelease((CUmemGenericAllocationHandle)handle);
        return r == CUDA_SUCCESS ? 0 : fail("cuMemRelease", r);
    }
    int map(uint64_t va, size_t bytes, uint64_t handle) override {
        CUresult r = pMap((CUdeviceptr)va, bytes, 0, (CUmemGenericAllocationHandle)handle, 0);
        return r == CUDA_SUCCESS ? 0 : fail("cuMemMap", r);
    }
    int set_access(uint64_t va, size_t bytes) override {
        CUmemAccessDesc a = {};
        a.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
        a.location.id = device;
        a.flags = CU_MEM_ACCESS_FLAGS_PROT_READWRITE;
        CUresult r = pSetAccess((CUdeviceptr)va, bytes, &a, 1);
        return r == CUDA_SUCCESS ? 0 : fail("cuMemSetAccess", r);
    }
    int unmap(uint64_t va, size_t bytes) override {
        CUresult r = pUnmap((CUdeviceptr)va, bytes);
        return r == CUDA_SUCCESS ? 0 : fail("cuMemUnmap", r);
    }
};

// Bookkeeping-only backend: hands out fake addresses and handles, checks the calling discipline
// (no double map, no unmap of an unmapped page, no leak of handles).
struct MockBackend : PageBackend {
    uint64_t next_va = 0x7000000000ull, next_handle = 1;
    std::vector<std::pair<uint64_t, uint64_t>> mapped;   // (va, bytes)
    bool is_mock() const override { return true; }
    int granularity(size_t *g) override { *g = (size_t)2 << 20; return 0; }
    int reserve(size_t bytes, size_t align, uint64_t *va) override {
        if (align == 0) align = (size_t)2 << 20;
        next_va = (next_va + align - 1) / align * align;
        *va = next_va;
        next_va += bytes;
        return 0;
    }
    int free_va(uint64_t, size_t) override { return 0; }
    int create(size_t, uint64_t *handle) override { *handle = next_handle++; return 0; }
    int release(uint64_t) override { return 0; }
    int map(uint64_t va, size_t bytes, uint64_t) override {
        for (auto &m : mapped)
            if (va < m.first + m.second && m.first < va + bytes) { last_error = "mock: double map"; return 6; }
        mapped.push_back({va, bytes});
        return 0;
    }
    int set_access(uint64_t va, size_t bytes) override {   // the range must be covered by mapped pages, without a hole
        size_t covered = 0;
        for (auto &m : mapped)
            if (m.first >= va && m.first + m.second <= va + bytes) covered += m.second;
            else if (va < m.first + m.second && m.first < va + bytes) { last_error = "mock: set_access cuts a mapping"; return 6; }
        if (covered != bytes) { last_error = "mock: set_access over an unmapped hole"; return 6; }
        return 0;
    }
    int unmap(uint64_t va, size_t bytes) override {        // whole mappings only, and no hole in the range
        size_t covered = 0;
        for (auto &m : mapped)
            if (m.first >= va && m.first + m.second <= va + bytes) covered += m.second;
            else if (va < m.first + m.second && m.first < va + bytes) { last_error = "mock: unmap cuts a mapping"; return 6; }
        if (covered != bytes) { last_error = "mock: unmap of an unmapped range"; return 6; }
        for (size_t i = 0; i < mapped.size();)
            if (mapped[i].first >= va && mapped[i].first + mapped[i].second <= va + bytes) {
                mapped[i] = mapped.back();
                mapped.pop_back();
            } else {
                ++i;
            }
        return 0;
    }
};

}  // namespace

PageBackend *make_cuda_backend(int device, std::string *err) {
    CudaBackend *b = new CudaBackend();
    b->device = device;
    bool ok = load_entry("cuMemGetAllocationGranularity", &b->pGranularity, err) &&
              load_entry("cuMemAddressReserve", &b->pReserve, err) &&
              load_entry("cuMemAddressFree", &b->pAddrFree, err) && load_entry("cuMemCreate", &b->pCreate, err) &&
              load_entry("cuMemRelease", &b->pRelease, err) && load_entry("cuMemMap", &b->pMap, err) &&
              load_entry("cuMemSetAccess", &b->pSetAccess, err) && load_entry("cuMemUnmap", &b->pUnmap, err) &&
              load_entry("cuGetErrorString", &b->pErrStr, err);
    if (!ok) {
        delete b;
        return nullptr;
    }
    return b;
}

PageBackend *make_mock_backend() { return new MockBackend(); }

// ------------------------------------------------------------------------------------------------
// Physical memory pool
// ------------------------------------------------------------------------------------------------
int PagePool::prealloc(uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t h;
        if (max_pages && live >= max_pages) return 2;
        int rc = be->create(page_bytes, &h);
        if (rc) return rc;
        ++created_total;
        ++live;
        free_list.push_back(h);
    }
    return 0;
}

int PagePool::acquire(uint64_t *handle) {
    if (!free_list.empty()) {
        *handle = free_list.back();
        free_list.pop_back();
        return 0;
    }
    if (max_pages && live >= max_pages) {
        be->last_error = "page budget exhausted";
        return 2;
    }
    int rc = be->create(page_bytes, handle);
    if (rc) return rc;
    ++created_total;
    ++live;
    return 0;
}

int PagePool::trim() {
    int rc = 0;
    for (uint64_t h : free_list) {
        int r = be->release(h);
        if (r) rc = r;
        --live;
    }
    free_list.clear();
    return rc;
}

// ------------------------------------------------------------------------------------------------
// Expert memory manager of one virtual weight tensor
// ------------------------------------------------------------------------------------------------
int VirtualTensor::init(PageBackend *be_, PagePool *pool_, size_t expert_bytes_, size_t n_slots_) {
    be = be_;
    pool = pool_;
    expert_bytes = expert_bytes_;
    n_slots = n_slots_;
    size_t page = pool->page_bytes;
    va_bytes = (expert_bytes * n_slots + page - 1) / page * page;
    int rc = be->reserve(va_bytes, page, &base);
    if (rc) return rc;
    refcnt.assign(va_bytes / page, 0);
    handle.assign(va_bytes / page, 0);
    pages_mapped = 0;
    return 0;
}

void VirtualTensor::destroy() {
    if (!be || !va_bytes) return;
    size_t page = pool->page_bytes;
    for (size_t p = 0; p < refcnt.size(); ++p)
        if (refcnt[p]) {
            be->unmap(base + p * page, page);
            pool->give_back(handle[p]);
            refcnt[p] = 0;
        }
    pages_mapped = 0;
    be->free_va(base, va_bytes);
    va_bytes = 0;
}

bool VirtualTensor::slot_mapped(size_t slot) const {
    size_t page = pool->page_bytes;
    size_t p0 = slot * expert_bytes / page, p1 = ((slot + 1) * expert_bytes - 1) / page;
    for (size_t p = p0; p <= p1; ++p)
        if (!refcnt[p]) return false;
    return true;
}

// Calls f(first_page, n_pages) for every maximal run of consecutive page indices in the ascending list `pages`.
template <class F>
static int for_each_run(const std::vector<size_t> &pages, F f) {
    for (size_t i = 0; i < pages.size();) {
        size_t j = i + 1;
        while (j < pages.size() && pages[j] == pages[j - 1] + 1) ++j;
        int rc = f(pages[i], j - i);
        if (rc) return rc;
        i = j;
    }
    return 0;
}

int VirtualTensor::map_slots(size_t first, size_t n) {
    size_t page = pool->page_bytes;
    std::vector<size_t> fresh;                 // pages mapped by this call, ascending
    for (size_t s = first; s < first + n; ++s) {
        size_t p0 = s * expert_bytes / page, p1 = ((s + 1) * expert_bytes - 1) / page;
        for (size_t p = p0; p <= p1; ++p) {
            if (refcnt[p] == 0) {
                uint64_t h;
                int rc = pool->acquire(&h);
                if (!rc) {
                    rc = be->map(base + p * page, page, h);
                    if (rc) pool->give_back(h);
                }
                if (rc) {   // undo: this expert's pages before p, then the experts before s
                    for (size_t q = p0; q < p; ++q)
                        if (--refcnt[q] == 0) { be->unmap(base + q * page, page); pool->give_back(handle[q]); --pages_mapped; }
                    unmap_slots(first, s - first);
                    return rc;
                }
                handle[p] = h;
                ++pages_mapped;
                fresh.push_back(p);
            }
            ++refcnt[p];
        }
    }
    // access rights once per run of new pages (an adapter's pages are one run, or two around a shared boundary page)
    int rc = for_each_run(fresh, [&](size_t p, size_t len) { return be->set_access(base + p * page, len * page); });
    if (rc) unmap_slots(first, n);
    return rc;
}

void VirtualTensor::unmap_slots(size_t first, size_t n) {
    size_t page = pool->page_bytes;
    std::vector<size_t> dead;                  // pages no live expert touches any more, ascending
    for (size_t s = first; s < first + n; ++s) {
        size_t p0 = s * expert_bytes / page, p1 = ((s + 1) * expert_bytes - 1) / page;
        for (size_t p = p0; p <= p1; ++p) {
            if (refcnt[p] == 0) continue;
            if (--refcnt[p] == 0) dead.push_back(p);
        }
    }
    for_each_run(dead, [&](size_t p, size_t len) {
        be->unmap(base + p * page, len * page);
        return 0;
    });
    for (size_t p : dead) {
        pool->give_back(handle[p]);
        --pages_mapped;
    }
}

}  // namespace ew
