"""Helpers shared by the GPU parity tests: error metrics, guard-banded device
buffers and host->device marshalling.  No operator arithmetic lives here."""
import numpy as np
import torch

GUARD_BYTES = 4096
_GUARD_WORD = 0x7FC0DEAD  # a quiet-NaN bit pattern


def max_rel(g, o) -> float:
    """Element-wise max |g - o| / |o| (for outputs with no cancellation, e.g. softmax)."""
    g, o = np.asarray(g, dtype=np.float64), np.asarray(o, dtype=np.float64)
    return float(np.max(np.abs(g - o) / np.abs(o))) if o.size else 0.0


def max_rel_floored(g, o) -> float:
    """max |g - o| / max(|o|, tau), tau = RMS of the oracle tensor: the relative
    error of outputs whose last step is an addition (the floor is the size of the
    summands; pure element-wise relative error is unbounded where they cancel)."""
    g, o = np.asarray(g, dtype=np.float64), np.asarray(o, dtype=np.float64)
    if not o.size:
        return 0.0
    tau = float(np.sqrt(np.mean(o * o)))
    return float(np.max(np.abs(g - o) / np.maximum(np.abs(o), tau)))


class Guarded:
    """A device tensor carved out of a larger allocation whose first and last
    4 KiB hold a NaN pattern; ``check()`` asserts nothing wrote outside."""

    def __init__(self, shape, dtype, device="cuda"):
        esize = torch.empty((), dtype=dtype).element_size()
        n = int(np.prod(shape))
        body = (n * esize + 15) // 16 * 16
        self._raw = torch.empty(GUARD_BYTES * 2 + body, dtype=torch.uint8, device=device)
        self._raw.view(torch.int32).fill_(_GUARD_WORD)
        self._body = body
        self.t = self._raw[GUARD_BYTES:GUARD_BYTES + n * esize].view(dtype).view(*shape)

    def check(self):
        w = self._raw.view(torch.int32)
        g = GUARD_BYTES // 4
        tail = w[g + self._body // 4:]
        assert bool((w[:g] == _GUARD_WORD).all()), "write before the buffer"
        assert bool((tail == _GUARD_WORD).all()), "write past the buffer"


def dev_f32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def dev_bf16(bits) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bfloat16 tensor (bit copy)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def host(t: torch.Tensor) -> np.ndarray:
    """CUDA tensor -> float64 numpy (exact widening)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
