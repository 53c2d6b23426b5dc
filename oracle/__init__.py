"""CPU oracle for the attention-JVP path.  Test infrastructure only: nothing in the product
package imports this; tests, the smoke check and the benchmark's CPU-baseline leg do."""
