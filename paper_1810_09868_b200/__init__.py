"""VGG19 forward / backward pass for NVIDIA B200 (sm_100a) behind a C ABI.

`binding` mirrors include/vgg19_b200.h one to one.  `Net` is a small
convenience holder: it creates a handle and lets torch allocate the device
workspace (torch is used for device memory and streams only).
"""
from __future__ import annotations

from . import binding
from .binding import *  # noqa: F401,F403


class Net:
    """Owns a vgg19 handle and its torch-allocated workspace."""

    def __init__(self, height, width, batch_max, dtype, params=None, seed=0, flags=0, mode=binding.VGG19_MODE_BACKWARD,
                 host_io=False, device="cuda:0"):
        import torch
        self._torch = torch
        self.height, self.width, self.batch_max, self.dtype = height, width, batch_max, dtype
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            if params is None:
                self.handle = binding.vgg19_create(height, width, batch_max, dtype, seed, flags)
            else:
                self.handle = binding.vgg19_create_from_params(height, width, batch_max, dtype, params, flags)
        self.n_tensors, self.n_params = binding.vgg19_param_count(self.handle)
        nbytes = binding.vgg19_workspace_bytes(self.handle, batch_max, mode)
        if host_io:
            nbytes += binding.vgg19_io_bytes(self.handle, batch_max, mode)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        binding.vgg19_bind_workspace(self.handle, self.workspace, nbytes)

    @property
    def act_dtype(self):
        return self._torch.bfloat16 if self.dtype == binding.VGG19_BF16 else self._torch.float32

    def forward(self, images, logits=None, probs=None, stream=None):
        torch = self._torch
        B = images.shape[0]
        if logits is None:
            logits = torch.empty(B, 1000, dtype=torch.float32, device=self.device)
        stream = stream or torch.cuda.current_stream(self.device)
        binding.vgg19_forward(self.handle, images, B, logits, probs, stream)
        return logits

    def backward(self, images, labels, grads=None, loss=None, logits=None, stream=None):
        torch = self._torch
        B = images.shape[0]
        if grads is None:
            grads = torch.empty(self.n_params, dtype=torch.float32, device=self.device)
        if loss is None:
            loss = torch.empty(1, dtype=torch.float32, device=self.device)
        stream = stream or torch.cuda.current_stream(self.device)
        binding.vgg19_backward(self.handle, images, labels, B, grads, loss, logits, stream)
        return grads, loss

    def sgd_step(self, grads, lr, stream=None):
        """parameters <- parameters - lr * grads, on the device, with every derived filter copy rebuilt."""
        binding.vgg19_sgd_step(self.handle, grads, lr, stream or self._torch.cuda.current_stream(self.device))

    def train_step(self, images, labels, lr, loss=None, stream=None):
        """Forward + backward + update as one recorded device program (workspace of VGG19_MODE_TRAIN)."""
        stream = stream or self._torch.cuda.current_stream(self.device)
        binding.vgg19_train_step(self.handle, images, labels, images.shape[0], lr, loss, stream)

    def saved_tensor(self, batch, mode, index):
        """View of a stored activation inside the workspace (no copy)."""
        off, dims = binding.vgg19_saved_tensor(self.handle, batch, mode, index)
        n = 1
        for d in dims:
            n *= d
        elt = 2 if self.dtype == binding.VGG19_BF16 else 4
        return self.workspace[off:off + n * elt].view(self.act_dtype).view(*dims)

    def param_slices(self):
        """[(offset, dims)] of the 38 tensors in the flat parameter buffer."""
        return [binding.vgg19_param_info(self.handle, i) for i in range(self.n_tensors)]

    def sync_status(self, stream=None):
        return binding.vgg19_sync_status(self.handle, stream or self._torch.cuda.current_stream(self.device))

    def close(self):
        if getattr(self, "handle", None):
            binding.vgg19_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
