// Virtual-memory-assisted expert weight management (Section 4.2 of the paper), host side.
//
//   PageBackend    the five primitives of Table 2 (reserve VA, create/free physical pages, map, unmap)
//                  either on the CUDA driver's virtual memory API or as a pure bookkeeping mock
//   PagePool       the per-device physical memory pool: fixed-size pages, pre-allocated, handed out at
//                  load time, returned on eviction and reused
//   VirtualTensor  the expert memory manager of one virtual weight tensor: slot -> byte range -> pages,
//                  with a reference count per page so that a page straddling two neighbouring
//                  adapters is mapped once (sub-page allocation)
#pragma once
#include <cstddef>
#include <cstdint>
#include <string>
#include <vector>

namespace ew {

struct PageBackend {
    virtual ~PageBackend() {}
    virtual bool is_mock() const = 0;
    virtual int granularity(size_t *g) = 0;
    virtual int reserve(size_t bytes, size_t align, uint64_t *va) = 0;
    virtual int free_va(uint64_t va, size_t bytes) = 0;
    virtual int create(size_t bytes, uint64_t *handle) = 0;
    virtual int release(uint64_t handle) = 0;
    virtual int map(uint64_t va, size_t bytes, uint64_t handle) = 0;   // map one page; not accessible yet
    // make a fully mapped range (any number of neighbouring pages) readable and writable: one driver call per run of
    // pages, because the call's cost hardly depends on the size of the range
    virtual int set_access(uint64_t va, size_t bytes) = 0;
    virtual int unmap(uint64_t va, size_t bytes) = 0;                  // a range made of whole mapped pages
    std::string last_error;
};

// device >= 0: CUDA driver backend (entry points fetched at run time, so the library loads on a
// machine without a driver); device < 0: mock.
PageBackend *make_cuda_backend(int device, std::string *err);
PageBackend *make_mock_backend();

struct PagePool {
    PageBackend *be = nullptr;
    size_t page_bytes = 0;
    uint64_t max_pages = 0;          // 0 = unlimited
    uint64_t created_total = 0;      // pages ever created
    uint64_t live = 0;               // created and not yet released to the driver
    std::vector<uint64_t> free_list;

    int prealloc(uint64_t n);
    int acquire(uint64_t *handle);   // 0 ok, 2 out of memory / over budget, 6 driver error
    void give_back(uint64_t handle) { free_list.push_back(handle); }
    int trim();
};

struct VirtualTensor {
    PageBackend *be = nullptr;
    PagePool *pool = nullptr;
    uint64_t base = 0;               // base_addr of the reserved range
    size_t expert_bytes = 0;         // expert_size of this stacked linear
    size_t n_slots = 0;
    size_t va_bytes = 0;
    std::vector<uint32_t> refcnt;    // per page: live experts whose bytes intersect it
    std::vector<uint64_t> handle;    // per page: physical page mapped there (valid when refcnt > 0)
    uint64_t pages_mapped = 0;

    int init(PageBackend *be, PagePool *pool, size_t expert_bytes, size_t n_slots);
    void destroy();
    // start_addr = base_addr + slot * expert_size (Section 4.2)
    uint64_t slot_addr(size_t slot) const { return base + (uint64_t)slot * expert_bytes; }
    // back slots [first, first+n) with pages; all-or-nothing
    int map_slots(size_t first, size_t n);
    void unmap_slots(size_t first, size_t n);
    bool slot_mapped(size_t slot) const;
};

}  // namespace ew
