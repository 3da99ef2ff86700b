"""CPU oracle for the DHQ forward path.  Test infrastructure only: nothing in the product
package imports this, and this package imports nothing from the product."""
