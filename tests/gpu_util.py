"""Helpers shared by the GPU parity tests: moving seeded inputs to the device and calling the C-ABI binding."""
import numpy as np
import torch

from paper_2511_13732_b200 import binding


def logits_to_device(a: np.ndarray, device="cuda"):
    """float32 array -> float32 tensor; uint16 bf16 bit patterns -> bfloat16 tensor (same bits)."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def make_handle(groups, slices_hint=0, weights=None):
    return binding.Groups(groups.V, groups.group_ptr, groups.group_tok, groups.tok_degree, weights=weights,
                          slices_hint=slices_hint)


def run_verify(batch, handle, mode=0):
    tl, dl = logits_to_device(batch.target_logits), logits_to_device(batch.draft_logits)
    x = torch.from_numpy(batch.draft_tokens).cuda()
    u = torch.from_numpy(batch.uniforms).cuda()
    n, tok, grp, flg = binding.pcg_verify(tl, dl, x, handle, u, batch.temperature, mode=mode)
    torch.cuda.synchronize()
    return n.cpu().numpy(), tok.cpu().numpy(), grp.cpu().numpy(), flg.cpu().numpy()


def run_oracle(oracle, batch, groups, weights=None):
    return oracle.verify(batch.target_logits, batch.draft_logits, batch.draft_tokens, groups.group_ptr,
                         groups.group_tok, groups.tok_degree, batch.uniforms, batch.temperature, weights=weights,
                         threads=0)


def library_candidate_order(V: int, logits: np.ndarray) -> np.ndarray:
    """The order in which pcg_verify_thinning's candidate draw walks the tokens, built here from the rule its
    header states: ascending ((t div W) mod 128, t) with W = 16 bytes / bytes per logit.  The oracle takes the
    order as an input; nothing of it is built into the oracle."""
    W = 16 // logits.dtype.itemsize
    t = np.arange(V)
    return np.lexsort((t, (t // W) % 128)).astype(np.int32)
