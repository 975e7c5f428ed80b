"""Convenience wrapper: owns a graph handle and runs it on torch CUDA tensors.

torch is used for device memory and streams only.
"""
from __future__ import annotations

from . import binding as B


class FusedGraph:
    def __init__(self, spec: str, device: int = 0, schedule: str | None = None, handle=None):
        self.handle = handle if handle is not None else B.hct_graph_create_scheduled(spec, device, schedule)
        self.device = device
        self.n_in = B.hct_graph_num_inputs(self.handle)
        self.n_out = B.hct_graph_num_outputs(self.handle)
        self.inputs = [B.hct_graph_tensor_info(self.handle, False, i) for i in range(self.n_in)]
        self.outputs = [B.hct_graph_tensor_info(self.handle, True, i) for i in range(self.n_out)]
        self.input_nhwc = [B.hct_graph_input_layout(self.handle, i) == 1 for i in range(self.n_in)]
        self.output_nhwc = [B.hct_graph_output_layout(self.handle, i) == 1 for i in range(self.n_out)]
        self.workspace_bytes = B.hct_graph_workspace_bytes(self.handle)
        self._ws = None

    @classmethod
    def autotuned(cls, spec: str, inputs, device: int = 0, max_trials: int = 16, workspace_bytes: int | None = None):
        """Measures candidate schedules on `inputs` (torch CUDA tensors in spec order) and keeps the fastest.
        Scratch outputs and a workspace are allocated here for the measurement (torch memory only)."""
        import torch
        probe = cls(spec, device)
        outs = probe.alloc_outputs()
        # room for every candidate's scratch plus the 160 MB the trials overwrite between runs to evict L2
        ws_bytes = workspace_bytes if workspace_bytes is not None else 2 * probe.workspace_bytes + (64 << 20) + (160 << 20)
        ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device=f"cuda:{device}")
        ws_ptr = (ws.data_ptr() + 255) // 256 * 256
        stream = torch.cuda.current_stream(device).cuda_stream
        probe.close()
        h = B.hct_graph_autotune(spec, device, [t.data_ptr() for t in inputs], [t.data_ptr() for t in outs], ws_ptr, ws_bytes, stream,
                                 max_trials)
        return cls(spec, device, handle=h)

    @property
    def schedule(self) -> str:
        return B.hct_graph_schedule(self.handle)

    # -- queries
    @property
    def plan(self) -> str:
        return B.hct_graph_plan_text(self.handle)

    @property
    def num_kernels(self) -> int:
        return B.hct_graph_num_kernels(self.handle)

    def cost(self):
        return B.hct_graph_cost(self.handle)

    def kernel_source(self, i: int) -> str:
        return B.hct_graph_kernel_source(self.handle, i)

    # -- execution on torch tensors
    def alloc_outputs(self):
        import torch
        outs = []
        for (_, dtype, shape), nhwc in zip(self.outputs, self.output_nhwc):
            # an output declared nhwc is a [N,C,H,W] tensor in torch's channels-last memory format
            outs.append(torch.empty(shape, dtype=torch.bfloat16 if dtype == B.HCT_BF16 else torch.float32, device=f"cuda:{self.device}",
                                    memory_format=torch.channels_last if nhwc else torch.contiguous_format))
        return outs

    def workspace(self):
        import torch
        if self._ws is None and self.workspace_bytes:
            self._ws = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=f"cuda:{self.device}")
        return self._ws

    def run(self, inputs, outputs=None, stream=None):
        """inputs: torch CUDA tensors in spec order.  Returns the output tensors.  Does not synchronise."""
        import torch
        if outputs is None:
            outputs = self.alloc_outputs()
        for t, (name, dtype, shape), nhwc in zip(inputs, self.inputs, self.input_nhwc):
            want = torch.bfloat16 if dtype == B.HCT_BF16 else torch.float32
            # an input declared nhwc is passed as a [N,C,H,W] tensor in torch's channels-last memory format
            dense = t.is_contiguous(memory_format=torch.channels_last) if nhwc else t.is_contiguous()
            if tuple(t.shape) != tuple(shape) or t.dtype != want or not dense or not t.is_cuda:
                raise ValueError(f"input {name}: expected {'channels-last' if nhwc else 'contiguous'} CUDA {want} tensor of shape {shape}")
        ws = self.workspace()
        ws_ptr = 0
        if ws is not None:
            ws_ptr = (ws.data_ptr() + 255) // 256 * 256
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        B.hct_graph_run(self.handle, [t.data_ptr() for t in inputs], [t.data_ptr() for t in outputs], ws_ptr, self.workspace_bytes,
                        s.cuda_stream)
        return outputs

    def status(self):
        B.hct_graph_status(self.handle)

    def close(self):
        if self.handle is not None:
            B.hct_graph_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
