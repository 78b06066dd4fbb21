"""CPU oracle of the EventGraD communication step.  TEST INFRASTRUCTURE ONLY: imported by
``tests/``, by ``__graft_entry__.smoke()`` and by ``bench.py``'s CPU-baseline legs; the CUDA
package never imports it."""
