"""Token-sharded tensors in one address range (CUDA virtual memory management, driver API).

The head-sharded sequence-parallel scheme (Section 4.1 of the paper) keeps q, k, v, o as [T, H, d] with
the T tokens split over the p ranks of a group, while attention needs all tokens of some heads.  Instead of
re-sharding with an all-to-all, every rank maps its own slice and its peers' slices, slice after slice,
into ONE virtual address range; the attention kernels then run on a group of heads of that range
(dcp_varlen_attn_fwd_strided / _bwd_strided) and fetch each tile from wherever it lives, with plain TMA
loads, when they need it.

A slice is one physical allocation (cuMemCreate) on its owner's GPU, exportable as a POSIX file
descriptor; peers import it (cuMemImportFromShareableHandle) and map it (cuMemMap) at the slice's offset
of their own range.  Slices must be whole allocation granules (2 MB on this hardware), so slice boundaries
fall on multiples of `tokens_per_granule`.

Only plumbing lives here: no arithmetic of the method.  On one GPU the same code runs with the p slices
all on that GPU (p "virtual ranks"), which is how it is tested.
"""
from __future__ import annotations

import math
import socket
from typing import List, Optional, Sequence, Tuple


def _drv():
    from cuda.bindings import driver
    return driver


def _ok(res, what: str):
    """cuda-python returns (CUresult, values...); raise unless CUDA_SUCCESS and hand back the values."""
    drv = _drv()
    err, rest = res[0], res[1:]
    if err != drv.CUresult.CUDA_SUCCESS:
        raise RuntimeError(f"{what} failed: {err}")
    return None if not rest else rest[0] if len(rest) == 1 else rest


def _alloc_prop(device: int):
    drv = _drv()
    prop = drv.CUmemAllocationProp()
    prop.type = drv.CUmemAllocationType.CU_MEM_ALLOCATION_TYPE_PINNED
    prop.location.type = drv.CUmemLocationType.CU_MEM_LOCATION_TYPE_DEVICE
    prop.location.id = device
    prop.requestedHandleTypes = drv.CUmemAllocationHandleType.CU_MEM_HANDLE_TYPE_POSIX_FILE_DESCRIPTOR
    return prop


def granularity(device: int) -> int:
    """Bytes every slice allocation must be a multiple of."""
    drv = _drv()
    return int(_ok(drv.cuMemGetAllocationGranularity(
        _alloc_prop(device), drv.CUmemAllocationGranularity_flags.CU_MEM_ALLOC_GRANULARITY_MINIMUM),
        "cuMemGetAllocationGranularity"))


def token_slices(total_tokens: int, p: int, row_bytes: int, gran: int) -> List[Tuple[int, int]]:
    """Contiguous token ranges of the p ranks whose byte sizes are whole granules (the last range takes what
    is left and is padded up by its owner).  Ranges are as even as the granule allows; trailing ranks may
    be empty when there are fewer granules than ranks."""
    if p < 1 or total_tokens < 0 or row_bytes < 1 or gran < 1:
        raise ValueError("need p >= 1, total_tokens >= 0, row_bytes >= 1, gran >= 1")
    tokens_per_granule = gran // math.gcd(gran, row_bytes)
    n_gran = -(-total_tokens // tokens_per_granule)
    base, extra = divmod(n_gran, p)
    out, start = [], 0
    for r in range(p):
        n = (base + (1 if r < extra else 0)) * tokens_per_granule
        end = min(start + n, total_tokens)
        out.append((start, end))
        start = end
    return out


class Slice:
    """One physical allocation on `device`, `nbytes` long (a whole number of granules)."""

    def __init__(self, nbytes: int, device: int, handle=None):
        drv = _drv()
        self.nbytes, self.device = int(nbytes), int(device)
        self.handle = handle if handle is not None else _ok(drv.cuMemCreate(self.nbytes, _alloc_prop(device), 0), "cuMemCreate")

    def export_fd(self) -> int:
        drv = _drv()
        return int(_ok(drv.cuMemExportToShareableHandle(
            self.handle, drv.CUmemAllocationHandleType.CU_MEM_HANDLE_TYPE_POSIX_FILE_DESCRIPTOR, 0),
            "cuMemExportToShareableHandle"))

    @staticmethod
    def import_fd(fd: int, nbytes: int, device: int) -> "Slice":
        drv = _drv()
        handle = _ok(drv.cuMemImportFromShareableHandle(
            fd, drv.CUmemAllocationHandleType.CU_MEM_HANDLE_TYPE_POSIX_FILE_DESCRIPTOR), "cuMemImportFromShareableHandle")
        return Slice(nbytes, device, handle)

    def release(self):
        if self.handle is not None:
            _drv().cuMemRelease(self.handle)
            self.handle = None


class _Cai:
    def __init__(self, ptr: int, nbytes: int):
        self.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (ptr, False), "version": 2}


class StitchedRange:
    """Slices mapped back to back into one reserved address range, readable and writable from `device`."""

    def __init__(self, slices: Sequence[Slice], device: int):
        drv = _drv()
        self.slices, self.device = list(slices), int(device)
        self.nbytes = sum(s.nbytes for s in self.slices)
        gran = granularity(device)
        self.ptr = int(_ok(drv.cuMemAddressReserve(self.nbytes, gran, 0, 0), "cuMemAddressReserve"))
        off = 0
        for s in self.slices:
            if s.nbytes:
                _ok(drv.cuMemMap(self.ptr + off, s.nbytes, 0, s.handle, 0), "cuMemMap")
            off += s.nbytes
        acc = drv.CUmemAccessDesc()
        acc.location.type = drv.CUmemLocationType.CU_MEM_LOCATION_TYPE_DEVICE
        acc.location.id = self.device
        acc.flags = drv.CUmemAccess_flags.CU_MEM_ACCESS_FLAGS_PROT_READWRITE
        _ok(drv.cuMemSetAccess(self.ptr, self.nbytes, [acc], 1), "cuMemSetAccess")

    def tensor(self, shape, dtype):
        """A torch view of the start of the range (it does not own the memory: keep this object alive)."""
        import torch
        n = int(math.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        if n > self.nbytes:
            raise ValueError("shape exceeds the mapped range")
        raw = torch.as_tensor(_Cai(self.ptr, self.nbytes), device=f"cuda:{self.device}")
        return raw[:n].view(dtype).view(*shape)

    def close(self):
        drv = _drv()
        if self.ptr:
            drv.cuMemUnmap(self.ptr, self.nbytes)
            drv.cuMemAddressFree(self.ptr, self.nbytes)
            self.ptr = 0


def slice_bytes(ranges: Sequence[Tuple[int, int]], row_bytes: int, gran: int) -> List[int]:
    """Allocation size of each token range: its bytes rounded up to whole granules (only the last non-empty
    range can need rounding)."""
    return [-(-((b - a) * row_bytes) // gran) * gran for a, b in ranges]


# ---- passing file descriptors between the ranks of one node (POSIX fds are per process) ------------------------------
def send_fds(sock: socket.socket, fds: Sequence[int]) -> None:
    """One descriptor per message (each with one payload byte), on the socket itself so that its timeout holds."""
    for fd in fds:
        socket.send_fds(sock, [b"f"], [fd])


def recv_fds(sock: socket.socket, n: int) -> List[int]:
    out = []
    for _ in range(n):
        msg, fds, _flags, _addr = socket.recv_fds(sock, 1, 1)
        if msg != b"f" or len(fds) != 1:
            raise ConnectionError("peer closed the socket before sending its descriptor")
        out.append(fds[0])
    return out


def stitched_tensors_local(total_tokens: int, n_heads: int, head_dim: int, p: int, device: int, n_tensors: int,
                           dtype=None):
    """n_tensors token-sharded [T, H, d] tensors whose p slices are separate allocations on ONE device: the
    single-GPU stand-in for a sequence-parallel group (p virtual ranks).  Returns (tensors, ranges, keepalive)."""
    import torch
    dtype = torch.bfloat16 if dtype is None else dtype
    torch.zeros(1, device=f"cuda:{device}")              # make sure the device's context exists and is current
    row_bytes = n_heads * head_dim * torch.empty((), dtype=dtype).element_size()
    gran = granularity(device)
    ranges = token_slices(total_tokens, p, row_bytes, gran)
    sizes = slice_bytes(ranges, row_bytes, gran)
    tensors, keep = [], []
    for _ in range(n_tensors):
        slices = [Slice(n, device) for n in sizes if n > 0]
        rng = StitchedRange(slices, device)
        keep.append(rng)
        tensors.append(rng.tensor((total_tokens, n_heads, head_dim), dtype))
    return tensors, ranges, keep


def exchange_fds(rank: int, p: int, my_fds: Sequence[int], socket_dir: str, tag: str, timeout: float = 60.0
                 ) -> List[Optional[List[int]]]:
    """Every rank of one node hands its file descriptors to every other rank.  Rank r listens on a Unix
    socket `socket_dir/tag.r`, connects to each peer's, sends (its rank, its descriptors) and receives the
    same from p - 1 peers.  Returns, per rank, the descriptors as valid in THIS process (None for itself).
    All ranks must call this with the same p, tag and number of descriptors."""
    import os
    import struct
    import time
    n = len(my_fds)
    path = os.path.join(socket_dir, f"{tag}.{rank}")
    if os.path.exists(path):
        os.unlink(path)
    server = socket.socket(socket.AF_UNIX, socket.SOCK_STREAM)
    server.bind(path)
    server.listen(p)
    server.settimeout(timeout)
    out: List[Optional[List[int]]] = [None] * p
    try:
        # connect to every peer (it may not be listening yet: retry until the deadline), send rank and descriptors
        conns = []
        for peer in range(p):
            if peer == rank:
                continue
            deadline = time.time() + timeout
            while True:
                c = socket.socket(socket.AF_UNIX, socket.SOCK_STREAM)
                try:
                    c.connect(os.path.join(socket_dir, f"{tag}.{peer}"))
                    break
                except (FileNotFoundError, ConnectionRefusedError):
                    c.close()
                    if time.time() > deadline:
                        raise TimeoutError(f"rank {rank}: peer {peer} never opened its socket")
                    time.sleep(0.01)
            c.sendall(struct.pack("<i", rank))
            send_fds(c, my_fds)
            conns.append(c)
        for _ in range(p - 1):
            c, _addr = server.accept()
            c.settimeout(timeout)
            (peer,) = struct.unpack("<i", c.recv(4, socket.MSG_WAITALL))
            out[peer] = recv_fds(c, n)
            c.close()
        for c in conns:
            c.close()
    finally:
        server.close()
        if os.path.exists(path):
            os.unlink(path)
    return out


def map_group(rank: int, p: int, sizes: Sequence[int], my_slices: Sequence[Slice], device: int, socket_dir: str, tag: str
              ) -> List[StitchedRange]:
    """For each of this rank's slices (one per token-sharded tensor, all `sizes[rank]` bytes): export it, swap
    descriptors with the p - 1 peers of the node, import theirs and map all p slices, in rank order, into one
    range per tensor on `device`.  sizes[r] = bytes of rank r's slice (0 = that rank holds no tokens)."""
    import os
    fds = [s.export_fd() for s in my_slices]
    theirs = exchange_fds(rank, p, fds, socket_dir, tag)
    ranges = []
    for t, mine in enumerate(my_slices):
        slices = []
        for r in range(p):
            if sizes[r] == 0:
                continue
            slices.append(mine if r == rank else Slice.import_fd(theirs[r][t], sizes[r], device))
        ranges.append(StitchedRange(slices, device))
    for fd in fds + [fd for peer in theirs if peer for fd in peer]:
        os.close(fd)                  # an imported or mapped allocation no longer needs its descriptor
    return ranges
