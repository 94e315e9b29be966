"""The failure path of the device-side bounded waits, made to happen without faulting or hanging anything.

The kernels that stage data through shared memory wait on copy barriers with a limit; when a wait runs out the
kernel records that in a device status word, returns, and the next synchronising call reports CDQ_ERR_TIMEOUT.
cdq_debug_expire_wait launches one small CTA that arms a barrier for bytes nobody sends and waits on it with that
same bounded wait (nothing is in flight, so the wait simply runs out); cdq_debug_set_device_status plants the
other flag from the host."""
import numpy as np
import pytest
import torch

from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import inputs
from tests.util import grid_of

pytestmark = pytest.mark.gpu

OK, CUDA, TIMEOUT = 0, 5, 6


def _small_layer():
    cfg = inputs.CONFIGS["C0"].scaled(d_in=64, d_out=16, n=256, seed=3)
    X, W = inputs.make_layer(cfg, device="cuda:0")
    g = grid_of(cfg)
    H = B.cdq_hessian(X)
    scale, zero, Q, _ = B.cdq_init_rtn(W, g)
    return cfg, H, W, g, scale, zero, Q


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable():
    lib = B.load()
    assert lib.cdq_last_device_status() == OK
    assert lib.cdq_debug_expire_wait(1 << 12, None) == OK       # enqueued; the kernel gives up after 4096 cycles
    assert lib.cdq_last_device_status() == TIMEOUT              # reported ...
    assert lib.cdq_last_device_status() == OK                   # ... once: reading clears the word
    cfg, H, W, g, scale, zero, Q = _small_layer()               # the context is intact
    stats = B.cdq_cd_solve(H, W, g, scale, zero, Q, 1)
    assert stats["committed"] >= 0 and lib.cdq_last_device_status() == OK


def test_a_synchronising_call_reports_the_timeout():
    lib = B.load()
    cfg, H, W, g, scale, zero, Q = _small_layer()
    Q0 = Q.clone()
    assert lib.cdq_debug_expire_wait(1 << 10, None) == OK
    with pytest.raises(B.CdqError) as err:                      # cdq_cd_solve with stats synchronises and reads the word
        B.cdq_cd_solve(H, W, g, scale, zero, Q, 1)
    assert err.value.status == TIMEOUT
    assert lib.cdq_last_device_status() == OK                   # cleared by the call that reported it
    Q.copy_(Q0)
    B.cdq_cd_solve(H, W, g, scale, zero, Q, 1)                  # and the next call is an ordinary one


def test_the_consistency_flag_maps_to_a_cuda_error_with_a_message():
    lib = B.load()
    assert lib.cdq_debug_set_device_status(2) == OK
    assert lib.cdq_last_device_status() == CUDA
    assert "out-of-range coordinate" in lib.cdq_last_error_detail().decode()
    assert lib.cdq_last_device_status() == OK
    assert lib.cdq_debug_set_device_status(1) == OK
    assert lib.cdq_last_device_status() == TIMEOUT
    assert lib.cdq_debug_set_device_status(3) == 1              # out of range: refused


def test_launch_counter_counts_kernels():
    lib = B.load()
    cfg, H, W, g, scale, zero, Q = _small_layer()
    torch.cuda.synchronize()
    before = lib.cdq_kernel_launches()
    B.cdq_layer_loss(H, W, g, scale, zero, Q)
    mid = lib.cdq_kernel_launches()
    assert mid - before >= 2          # residual, H E (+ reductions)
    lib.cdq_debug_expire_wait(1 << 10, None)
    assert lib.cdq_kernel_launches() == mid + 1
    assert lib.cdq_last_device_status() == TIMEOUT
