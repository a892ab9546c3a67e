"""Symmetric heap for the pull-mode call (Sec. 4.1: partial outputs and flags of all ranks are
reachable from every rank; Sec. 4.2: reducers read the peers' tiles themselves).

One process per rank.  Every rank allocates one segment, hands it to the other ranks as a file
descriptor, and maps all W segments into one address range at a uniform stride, so that
segment w starts at `base + w * stride` in every process: the layout `entwine_gemm_rs_pull`
asks for.  The memory comes from a backend:

* `VmmBackend`  - device memory through the CUDA virtual-memory API (shareable POSIX handles);
                  a peer's segment is peer-mapped memory of that rank's GPU;
* `MemfdBackend` - host memory (memfd + mmap): the same exchange and layout without a GPU, for
                  tests of the host logic.

File descriptors travel over Unix-domain sockets (SCM_RIGHTS); the socket paths and the
barriers go through `torch.distributed` (any backend; gloo in the tests).  Nothing here runs
on the hot path: the heap is set up once and reused by every call.
"""
from __future__ import annotations

import ctypes
import os
import socket
import tempfile
import threading


def _round_up(v: int, to: int) -> int:
    return (v + to - 1) // to * to


def exchange_fds(my_fd: int, rank: int, world: int, dist, group=None) -> list:
    """All-gather of one file descriptor per rank.  Returns W descriptors valid in this
    process; entry `rank` is `my_fd` itself.  `dist` is torch.distributed (initialised)."""
    tmp = tempfile.mkdtemp(prefix="entwine_heap_")
    path = os.path.join(tmp, f"r{rank}.sock")
    srv = socket.socket(socket.AF_UNIX, socket.SOCK_STREAM)
    srv.bind(path)
    srv.listen(world)
    srv.settimeout(60.0)
    errors = []

    def serve():
        try:
            for _ in range(world - 1):
                conn, _ = srv.accept()
                with conn:
                    socket.send_fds(conn, [b"f"], [my_fd])
        except Exception as e:  # reported by the caller's thread
            errors.append(e)

    th = threading.Thread(target=serve, daemon=True)
    th.start()
    paths = [None] * world
    dist.all_gather_object(paths, path, group=group)
    fds = [None] * world
    fds[rank] = my_fd
    try:
        for q in range(world):
            if q == rank:
                continue
            with socket.socket(socket.AF_UNIX, socket.SOCK_STREAM) as c:
                c.settimeout(60.0)
                c.connect(paths[q])
                _, got, _, _ = socket.recv_fds(c, 1, 1)
                if len(got) != 1:
                    raise RuntimeError(f"rank {q} sent no descriptor")
                fds[q] = got[0]
        th.join(60.0)
        if errors:
            raise errors[0]
        if th.is_alive():
            raise RuntimeError("a peer never fetched this rank's descriptor")
    finally:
        dist.barrier(group=group)
        srv.close()
        try:
            os.unlink(path)
            os.rmdir(tmp)
        except OSError:
            pass
    return fds


class MemfdBackend:
    """Host memory: anonymous files mapped at fixed addresses inside one reserved range."""
    name = "memfd"

    def __init__(self):
        self._libc = ctypes.CDLL(None, use_errno=True)
        self._libc.mmap.restype = ctypes.c_void_p
        self._libc.mmap.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                    ctypes.c_long]
        self._libc.munmap.argtypes = [ctypes.c_void_p, ctypes.c_size_t]
        self._reserved = []

    def granularity(self) -> int:
        return os.sysconf("SC_PAGE_SIZE")

    def create(self, size: int) -> int:
        fd = os.memfd_create("entwine_segment")
        os.ftruncate(fd, size)  # zero-filled
        return fd

    def reserve(self, total: int) -> int:
        PROT_NONE, MAP_PRIVATE, MAP_ANONYMOUS = 0, 0x02, 0x20
        base = self._libc.mmap(None, total, PROT_NONE, MAP_PRIVATE | MAP_ANONYMOUS, -1, 0)
        if base in (None, ctypes.c_void_p(-1).value):
            raise OSError(ctypes.get_errno(), "mmap (reserve)")
        self._reserved.append((base, total))
        return base

    def map(self, addr: int, size: int, fd: int, own: bool) -> None:
        PROT_RW, MAP_SHARED, MAP_FIXED = 0x1 | 0x2, 0x01, 0x10
        got = self._libc.mmap(addr, size, PROT_RW, MAP_SHARED | MAP_FIXED, fd, 0)
        if got != addr:
            raise OSError(ctypes.get_errno(), "mmap (map)")

    def finish(self, base: int, total: int) -> None:
        pass

    def zero(self, addr: int, size: int) -> None:
        ctypes.memset(addr, 0, size)

    def close(self) -> None:
        for base, total in self._reserved:
            self._libc.munmap(base, total)
        self._reserved = []


class VmmBackend:
    """Device memory of the current CUDA device through the virtual-memory API."""
    name = "cuda-vmm"

    def __init__(self, device: int | None = None):
        import torch
        from cuda.bindings import driver as drv
        self._drv = drv
        self.device = torch.cuda.current_device() if device is None else int(device)
        torch.zeros(1, device=f"cuda:{self.device}")  # the primary context is current from here on
        prop = drv.CUmemAllocationProp()
        prop.type = drv.CUmemAllocationType.CU_MEM_ALLOCATION_TYPE_PINNED
        prop.location.type = drv.CUmemLocationType.CU_MEM_LOCATION_TYPE_DEVICE
        prop.location.id = self.device
        prop.requestedHandleTypes = drv.CUmemAllocationHandleType.CU_MEM_HANDLE_TYPE_POSIX_FILE_DESCRIPTOR
        self._prop = prop
        self._fd_type = drv.CUmemAllocationHandleType.CU_MEM_HANDLE_TYPE_POSIX_FILE_DESCRIPTOR
        self._handles, self._mapped, self._reserved = [], [], []

    def _ck(self, res, what):
        err = res[0] if isinstance(res, tuple) else res
        if int(err) != 0:
            raise RuntimeError(f"{what}: CUDA driver error {int(err)}")
        if isinstance(res, tuple):
            return res[1] if len(res) == 2 else res[1:]
        return None

    def granularity(self) -> int:
        drv = self._drv
        return int(self._ck(drv.cuMemGetAllocationGranularity(
            self._prop, drv.CUmemAllocationGranularity_flags.CU_MEM_ALLOC_GRANULARITY_RECOMMENDED),
            "cuMemGetAllocationGranularity"))

    def create(self, size: int) -> int:
        drv = self._drv
        h = self._ck(drv.cuMemCreate(size, self._prop, 0), "cuMemCreate")
        self._handles.append(h)
        self._own = h
        return int(self._ck(drv.cuMemExportToShareableHandle(h, self._fd_type, 0), "cuMemExportToShareableHandle"))

    def reserve(self, total: int) -> int:
        ptr = self._ck(self._drv.cuMemAddressReserve(total, self.granularity(), 0, 0), "cuMemAddressReserve")
        self._reserved.append((int(ptr), total))
        return int(ptr)

    def map(self, addr: int, size: int, fd: int, own: bool) -> None:
        drv = self._drv
        if own:
            h = self._own
        else:
            h = self._ck(drv.cuMemImportFromShareableHandle(fd, self._fd_type), "cuMemImportFromShareableHandle")
            self._handles.append(h)
        self._ck(drv.cuMemMap(addr, size, 0, h, 0), "cuMemMap")
        self._mapped.append((addr, size))

    def finish(self, base: int, total: int) -> None:
        drv = self._drv
        acc = drv.CUmemAccessDesc()
        acc.location.type = drv.CUmemLocationType.CU_MEM_LOCATION_TYPE_DEVICE
        acc.location.id = self.device
        acc.flags = drv.CUmemAccess_flags.CU_MEM_ACCESS_FLAGS_PROT_READWRITE
        self._ck(drv.cuMemSetAccess(base, total, [acc], 1), "cuMemSetAccess")

    def zero(self, addr: int, size: int) -> None:
        self._ck(self._drv.cuMemsetD8(addr, 0, size), "cuMemsetD8")
        self._ck(self._drv.cuCtxSynchronize(), "cuCtxSynchronize")

    def close(self) -> None:
        drv = self._drv
        for addr, size in self._mapped:
            drv.cuMemUnmap(addr, size)
        for h in self._handles:
            drv.cuMemRelease(h)
        for base, total in self._reserved:
            drv.cuMemAddressFree(base, total)
        self._mapped, self._handles, self._reserved = [], [], []


class SymmetricHeap:
    """W segments at `base + w * stride`; segment `rank` is this process's own memory.

    segment_bytes: what `Plan.heap_bytes()[0]` reports (or more); the stride is that rounded up
    to the backend's granularity.  Collective over `group`: every rank must construct it."""

    def __init__(self, segment_bytes: int, rank: int, world: int, dist, backend, group=None):
        self.rank, self.world, self.backend = rank, world, backend
        self.stride = _round_up(_round_up(int(segment_bytes), 256), backend.granularity())
        own_fd = backend.create(self.stride)
        fds = exchange_fds(own_fd, rank, world, dist, group)
        self.base = backend.reserve(self.stride * world)
        for w in range(world):
            backend.map(self.base + w * self.stride, self.stride, fds[w], own=(w == rank))
        backend.finish(self.base, self.stride * world)
        for fd in fds:
            os.close(fd)
        backend.zero(self.segment(rank), self.stride)
        dist.barrier(group=group)  # every segment is zero before anyone's first call

    def segment(self, w: int) -> int:
        if not 0 <= w < self.world:
            raise IndexError(w)
        return self.base + w * self.stride

    def cuda_tensor(self, w: int, offset: int, nbytes: int):
        """uint8 torch view of part of segment w (VmmBackend only)."""
        import torch

        class _View:
            pass
        v = _View()
        v.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (self.segment(w) + offset, False),
                                      "version": 3}
        return torch.as_tensor(v, device=f"cuda:{self.backend.device}")

    def close(self) -> None:
        self.backend.close()
