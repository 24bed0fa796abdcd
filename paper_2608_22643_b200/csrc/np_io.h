// Record reads from a store file (Section 3.5: incoming IDs are sorted, adjacent IDs coalesced
// into contiguous ranges, the ranges submitted through io_uring on a file opened with O_DIRECT,
// a bounded number of reads in flight, completions landing in page-aligned pinned staging).
//
// Host code only.  One RecordReader belongs to one thread at a time.  Reads are queued in
// groups (a group = one part of the staging buffer); the caller queues a group, goes on to queue
// the next one, and waits for a group when it needs its bytes, so the device queue stays full
// across groups.  Where the kernel offers no io_uring (old kernel, seccomp), or when asked to,
// the same interface runs on blocking preads issued when a group is waited for.
#pragma once

#include <stddef.h>
#include <stdint.h>

#include <functional>
#include <string>
#include <vector>

namespace npi {

class RecordReader {
 public:
  static constexpr int kGroups = 8;               // group tags 0 .. kGroups-1
  static constexpr size_t kMaxRead = 1u << 20;    // longer ranges are cut into reads of this size
  static constexpr int kDefaultDepth = 256;       // reads in flight (the paper's queue depth)

  RecordReader() = default;
  ~RecordReader() { close(); }
  RecordReader(const RecordReader&) = delete;
  RecordReader& operator=(const RecordReader&) = delete;

  // depth > 0: io_uring with up to `depth` reads in flight; if the ring cannot be set up the
  // reader falls back to blocking reads and says why in `note`.  depth < 0: blocking reads.
  // `parallel` (may be empty) runs n independent jobs, possibly on several threads; the
  // blocking path uses it to overlap its preads.
  bool open(int fd, int depth, std::function<void(int, const std::function<void(int)>&)> parallel, std::string* note);
  void close();
  bool is_open() const { return fd_ >= 0; }
  bool uses_ring() const { return ring_fd_ >= 0; }
  int depth() const { return depth_; }

  // Queues the read of file bytes [off, off + len) into dst for group `tag`; cuts it into reads
  // of at most kMaxRead.  May block until the ring has room.  false: the submission failed
  // (errno-style code in last_error()); reads already queued stay queued.
  bool submit(void* dst, size_t len, uint64_t off, int tag);
  // Blocks until every read of the group has completed.  false: one of them failed.
  bool wait_group(int tag);
  // Blocks until nothing is in flight (every group).  Call before the buffers go away.
  bool drain();
  int last_error() const { return err_; }
  uint64_t reads_done() const { return reads_done_; }
  uint64_t bytes_done() const { return bytes_done_; }

 private:
  struct Req {
    char* dst;
    size_t len;
    uint64_t off;
    int tag;
  };
  bool ring_setup(int depth, std::string* note);
  bool ring_push(int slot);            // writes the SQE of reqs_[slot]
  bool ring_enter(unsigned to_submit, unsigned min_complete);
  void ring_reap();                    // consumes the completions that are there
  bool run_blocking(int tag);

  int fd_ = -1;
  int depth_ = 0;
  int err_ = 0;
  uint64_t reads_done_ = 0, bytes_done_ = 0;
  std::function<void(int, const std::function<void(int)>&)> parallel_;

  // io_uring state
  int ring_fd_ = -1;
  void* sq_ptr_ = nullptr;
  void* cq_ptr_ = nullptr;
  void* sqes_ = nullptr;
  size_t sq_len_ = 0, cq_len_ = 0, sqes_len_ = 0;
  unsigned *sq_head_ = nullptr, *sq_tail_ = nullptr, *sq_mask_ = nullptr, *sq_array_ = nullptr;
  unsigned *cq_head_ = nullptr, *cq_tail_ = nullptr, *cq_mask_ = nullptr;
  void* cqes_ = nullptr;
  unsigned unsubmitted_ = 0;           // SQEs written but not yet handed to the kernel
  int in_flight_ = 0;

  std::vector<Req> reqs_;              // one slot per read in flight (ring) / per queued read (blocking)
  std::vector<int> free_;              // free slots of reqs_ (ring)
  int outstanding_[kGroups] = {};
  bool failed_[kGroups] = {};
  std::vector<Req> queued_[kGroups];   // blocking path: reads waiting for wait_group
};

}  // namespace npi
