// Record reads from a store file through io_uring (raw system calls: the image has the kernel
// header but no liburing), with a blocking-pread fallback.  See np_io.h.  Host code only.
#include "np_io.h"

#include <errno.h>
#include <linux/io_uring.h>
#include <string.h>
#include <sys/mman.h>
#include <sys/syscall.h>
#include <unistd.h>

#include <algorithm>
#include <atomic>

namespace npi {

namespace {

int sys_io_uring_setup(unsigned entries, io_uring_params* p) { return (int)syscall(__NR_io_uring_setup, entries, p); }
int sys_io_uring_enter(int fd, unsigned to_submit, unsigned min_complete, unsigned flags) {
  return (int)syscall(__NR_io_uring_enter, fd, to_submit, min_complete, flags, nullptr, 0);
}

inline unsigned load_acquire(const unsigned* p) { return __atomic_load_n(p, __ATOMIC_ACQUIRE); }
inline void store_release(unsigned* p, unsigned v) { __atomic_store_n(p, v, __ATOMIC_RELEASE); }

// pread until the range is complete; 0 or an errno-style code
int pread_full(int fd, char* dst, size_t len, uint64_t off) {
  while (len > 0) {
    const ssize_t r = pread(fd, dst, len, (off_t)off);
    if (r < 0) {
      if (errno == EINTR) continue;
      return errno;
    }
    if (r == 0) return ENODATA;  // the file is shorter than the store it should hold
    dst += r;
    off += (uint64_t)r;
    len -= (size_t)r;
  }
  return 0;
}

}  // namespace

bool RecordReader::open(int fd, int depth, std::function<void(int, const std::function<void(int)>&)> parallel,
                        std::string* note) {
  close();
  if (fd < 0) {
    err_ = EBADF;
    return false;
  }
  fd_ = fd;
  parallel_ = std::move(parallel);
  err_ = 0;
  reads_done_ = bytes_done_ = 0;
  for (int g = 0; g < kGroups; ++g) {
    outstanding_[g] = 0;
    failed_[g] = false;
    queued_[g].clear();
  }
  if (depth == 0) depth = kDefaultDepth;
  depth_ = depth;
  if (depth > 0 && !ring_setup(depth, note)) depth_ = -1;  // blocking reads from here on
  return true;
}

void RecordReader::close() {
  if (fd_ < 0) return;
  drain();
  if (sqes_) munmap(sqes_, sqes_len_);
  if (cq_ptr_ && cq_ptr_ != sq_ptr_) munmap(cq_ptr_, cq_len_);
  if (sq_ptr_) munmap(sq_ptr_, sq_len_);
  if (ring_fd_ >= 0) ::close(ring_fd_);
  sqes_ = cq_ptr_ = sq_ptr_ = nullptr;
  ring_fd_ = -1;
  fd_ = -1;
  reqs_.clear();
  free_.clear();
  in_flight_ = 0;
  unsubmitted_ = 0;
}

bool RecordReader::ring_setup(int depth, std::string* note) {
  io_uring_params p;
  memset(&p, 0, sizeof(p));
  unsigned entries = 1;
  while ((int)entries < depth && entries < 4096) entries <<= 1;
  const int rfd = sys_io_uring_setup(entries, &p);
  if (rfd < 0) {
    if (note) *note = std::string("io_uring_setup: ") + strerror(errno) + "; blocking reads instead";
    return false;
  }
  sq_len_ = p.sq_off.array + p.sq_entries * sizeof(unsigned);
  cq_len_ = p.cq_off.cqes + p.cq_entries * sizeof(io_uring_cqe);
  const bool single = (p.features & IORING_FEAT_SINGLE_MMAP) != 0;
  if (single) sq_len_ = cq_len_ = std::max(sq_len_, cq_len_);
  sq_ptr_ = mmap(nullptr, sq_len_, PROT_READ | PROT_WRITE, MAP_SHARED | MAP_POPULATE, rfd, IORING_OFF_SQ_RING);
  if (sq_ptr_ == MAP_FAILED) sq_ptr_ = nullptr;
  if (sq_ptr_) {
    if (single) {
      cq_ptr_ = sq_ptr_;
    } else {
      cq_ptr_ = mmap(nullptr, cq_len_, PROT_READ | PROT_WRITE, MAP_SHARED | MAP_POPULATE, rfd, IORING_OFF_CQ_RING);
      if (cq_ptr_ == MAP_FAILED) cq_ptr_ = nullptr;
    }
  }
  sqes_len_ = p.sq_entries * sizeof(io_uring_sqe);
  if (sq_ptr_ && cq_ptr_) {
    sqes_ = mmap(nullptr, sqes_len_, PROT_READ | PROT_WRITE, MAP_SHARED | MAP_POPULATE, rfd, IORING_OFF_SQES);
    if (sqes_ == MAP_FAILED) sqes_ = nullptr;
  }
  if (!sq_ptr_ || !cq_ptr_ || !sqes_) {
    if (note) *note = std::string("io_uring mmap: ") + strerror(errno) + "; blocking reads instead";
    if (sqes_) munmap(sqes_, sqes_len_);
    if (cq_ptr_ && cq_ptr_ != sq_ptr_) munmap(cq_ptr_, cq_len_);
    if (sq_ptr_) munmap(sq_ptr_, sq_len_);
    sqes_ = cq_ptr_ = sq_ptr_ = nullptr;
    ::close(rfd);
    return false;
  }
  char* sq = static_cast<char*>(sq_ptr_);
  char* cq = static_cast<char*>(cq_ptr_);
  sq_head_ = reinterpret_cast<unsigned*>(sq + p.sq_off.head);
  sq_tail_ = reinterpret_cast<unsigned*>(sq + p.sq_off.tail);
  sq_mask_ = reinterpret_cast<unsigned*>(sq + p.sq_off.ring_mask);
  sq_array_ = reinterpret_cast<unsigned*>(sq + p.sq_off.array);
  cq_head_ = reinterpret_cast<unsigned*>(cq + p.cq_off.head);
  cq_tail_ = reinterpret_cast<unsigned*>(cq + p.cq_off.tail);
  cq_mask_ = reinterpret_cast<unsigned*>(cq + p.cq_off.ring_mask);
  cqes_ = cq + p.cq_off.cqes;
  ring_fd_ = rfd;
  depth_ = std::min<int>(depth, (int)p.sq_entries);
  reqs_.assign(depth_, Req{nullptr, 0, 0, 0});
  free_.clear();
  for (int i = depth_ - 1; i >= 0; --i) free_.push_back(i);
  in_flight_ = 0;
  unsubmitted_ = 0;
  return true;
}

bool RecordReader::ring_push(int slot) {
  const Req& r = reqs_[slot];
  const unsigned tail = *sq_tail_;  // only this thread writes the tail
  const unsigned idx = tail & *sq_mask_;
  io_uring_sqe* sqe = static_cast<io_uring_sqe*>(sqes_) + idx;
  memset(sqe, 0, sizeof(*sqe));
  sqe->opcode = IORING_OP_READ;
  sqe->fd = fd_;
  sqe->addr = (uint64_t)(uintptr_t)r.dst;
  sqe->len = (unsigned)r.len;
  sqe->off = r.off;
  sqe->user_data = (uint64_t)slot;
  sq_array_[idx] = idx;
  store_release(sq_tail_, tail + 1);
  ++unsubmitted_;
  return true;
}

bool RecordReader::ring_enter(unsigned to_submit, unsigned min_complete) {
  for (;;) {
    const int r = sys_io_uring_enter(ring_fd_, to_submit, min_complete, min_complete ? IORING_ENTER_GETEVENTS : 0);
    if (r >= 0) {
      unsubmitted_ -= std::min<unsigned>(unsubmitted_, (unsigned)r);
      return true;
    }
    if (errno == EINTR) continue;
    if (errno == EAGAIN || errno == EBUSY) {  // completions must be consumed first
      ring_reap();
      continue;
    }
    err_ = errno;
    return false;
  }
}

void RecordReader::ring_reap() {
  unsigned head = *cq_head_;
  const unsigned tail = load_acquire(cq_tail_);
  while (head != tail) {
    const io_uring_cqe* cqe = static_cast<const io_uring_cqe*>(cqes_) + (head & *cq_mask_);
    const int slot = (int)cqe->user_data;
    const int res = cqe->res;
    ++head;
    Req& r = reqs_[slot];
    if (res > 0 && (size_t)res < r.len) {
      // a short read: ask for the rest (the slot stays in flight)
      r.dst += res;
      r.off += (uint64_t)res;
      r.len -= (size_t)res;
      bytes_done_ += (uint64_t)res;
      ring_push(slot);
      continue;
    }
    if (res <= 0) {
      failed_[r.tag] = true;
      err_ = res < 0 ? -res : ENODATA;
    } else {
      bytes_done_ += (uint64_t)res;
      ++reads_done_;
    }
    --outstanding_[r.tag];
    --in_flight_;
    free_.push_back(slot);
  }
  store_release(cq_head_, head);
}

bool RecordReader::submit(void* dst, size_t len, uint64_t off, int tag) {
  if (fd_ < 0 || tag < 0 || tag >= kGroups) {
    err_ = EINVAL;
    return false;
  }
  char* p = static_cast<char*>(dst);
  while (len > 0) {
    const size_t n = std::min(len, kMaxRead);
    if (ring_fd_ < 0) {
      queued_[tag].push_back(Req{p, n, off, tag});
      ++outstanding_[tag];
    } else {
      while (free_.empty()) {  // the ring is full: hand over what is written and wait for one completion
        if (!ring_enter(unsubmitted_, 1)) return false;
        ring_reap();
      }
      const int slot = free_.back();
      free_.pop_back();
      reqs_[slot] = Req{p, n, off, tag};
      ++outstanding_[tag];
      ++in_flight_;
      ring_push(slot);
      // hand requests to the kernel in small batches: early ones start while later ones are written
      if (unsubmitted_ >= 16 && !ring_enter(unsubmitted_, 0)) return false;
    }
    p += n;
    off += n;
    len -= n;
  }
  return true;
}

bool RecordReader::run_blocking(int tag) {
  std::vector<Req>& q = queued_[tag];
  const int n = (int)q.size();
  std::atomic<int> first_err{0};
  auto job = [&](int i) {
    const int e = pread_full(fd_, q[i].dst, q[i].len, q[i].off);
    if (e) {
      int zero = 0;
      first_err.compare_exchange_strong(zero, e);
    }
  };
  if (parallel_ && n > 1) parallel_(n, job);
  else for (int i = 0; i < n; ++i) job(i);
  for (int i = 0; i < n; ++i) bytes_done_ += q[i].len;
  reads_done_ += (uint64_t)n;
  outstanding_[tag] -= n;
  q.clear();
  if (first_err.load()) {
    err_ = first_err.load();
    failed_[tag] = true;
  }
  return !failed_[tag];
}

bool RecordReader::wait_group(int tag) {
  if (fd_ < 0 || tag < 0 || tag >= kGroups) {
    err_ = EINVAL;
    return false;
  }
  if (ring_fd_ < 0) {
    const bool ok = run_blocking(tag);
    failed_[tag] = false;
    return ok;
  }
  if (unsubmitted_ && !ring_enter(unsubmitted_, 0)) return false;
  ring_reap();
  while (outstanding_[tag] > 0) {
    if (!ring_enter(unsubmitted_, 1)) return false;
    ring_reap();
  }
  const bool ok = !failed_[tag];
  failed_[tag] = false;
  return ok;
}

bool RecordReader::drain() {
  if (fd_ < 0) return true;
  bool ok = true;
  for (int g = 0; g < kGroups; ++g)
    if (outstanding_[g] > 0 || failed_[g]) ok = wait_group(g) && ok;
  return ok;
}

}  // namespace npi
